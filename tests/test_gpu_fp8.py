"""GPU parity with 8-bit (FP8 E4M3) caches: the append stores exactly the codes
of the oracle's quantiser (O6), the decode step attends over the dequantised
values like O1 / O2 on the logical history."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, attn_errors, f64

pytestmark = pytest.mark.gpu


class Fp8Stack:
    def __init__(self, L, B, Hq, Hkv, S, R, cap, scales, **kw):
        D = 128
        self.scales = torch.tensor(scales, dtype=torch.float32).cuda().contiguous()          # [L][2]
        self.shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, lt.LT_BF16, 0.0, kv_fp8=1, kv_scales=self.scales, **kw)
        mk = lambda n: [torch.zeros((B, Hkv, n, D), dtype=torch.uint8, device="cuda") for _ in range(L)]
        self.k_full, self.v_full, self.k_stream, self.v_stream = mk(cap), mk(cap), mk(S + R), mk(S + R)
        self.tables = lt.LayerTables(self.shape, self.k_full, self.v_full, self.k_stream, self.v_stream)
        self.ws = torch.empty(lt.workspace_bytes(self.shape), dtype=torch.uint8, device="cuda")
        lt.workspace_init(self.ws)
        self.seq_lens = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.mask = torch.zeros(L, dtype=torch.uint8, device="cuda")


@pytest.mark.parametrize("Hq,Hkv,S,R,lens,steps", [
    (8, 2, 4, 28, [300, 1, 31, 2047], 36),         # G = 4; the ring wraps; a chunk boundary is crossed
    (5, 1, 0, 16, [70, 15], 20),                   # G = 5, no sink
    (16, 2, 3, 9, [5, 0], 14),                     # G = 8, starts (almost) empty
    (32, 2, 4, 28, [300, 2047, 33], 36),           # G = 16: warp pairs on the byte path, ring wraps, chunk boundary
    (12, 1, 2, 12, [4200, 64], 6),                 # G = 12: the second warp of a pair serves four heads; several chunks
    (32, 1, 4, 28, [300, 2047, 33], 36),           # G = 32: four warps per tile on the byte path, ring wraps
    (20, 1, 0, 12, [4200, 64, 0], 6),              # G = 20: the third warp serves four heads, the fourth none; several chunks
])
def test_fp8_caches_append_codes_and_attention(Hq, Hkv, S, R, lens, steps):
    torch.manual_seed(33)
    g = np.random.default_rng(33)
    L, B, D = 3, len(lens), 128
    mask = np.array([0, 1, 0], dtype=np.uint8)
    cap = max(lens) + steps + 1
    scales = g.uniform(0.015, 0.04, size=(L, 2)).astype(np.float32)
    fus = Fp8Stack(L, B, Hq, Hkv, S, R, cap, scales)
    sep = Fp8Stack(L, B, Hq, Hkv, S, R, cap, scales)
    replays = [O.HybridReplay(mask, S, R) for _ in range(B)]
    codes_hist = [[None] * B for _ in range(L)]                                  # K codes of the logical history
    for l in range(L):
        hk = torch.randn(B, Hkv, max(lens), D).bfloat16()
        hv = torch.randn(B, Hkv, max(lens), D).bfloat16()
        kc, kval = O.quantize_e4m3(f64(hk), scales[l, 0])
        vc, vval = O.quantize_e4m3(f64(hv), scales[l, 1])
        for st in (fus, sep):
            st.k_full[l][:, :, :max(lens)] = torch.from_numpy(kc).cuda()
            st.v_full[l][:, :, :max(lens)] = torch.from_numpy(vc).cuda()
        for b, n in enumerate(lens):
            replays[b].load_prompt(l, kval[b, :, :n], vval[b, :, :n])
            codes_hist[l][b] = kc[b, :, :n]
    for st in (fus, sep):
        st.mask.copy_(torch.from_numpy(mask)); st.seq_lens.copy_(torch.tensor(lens, dtype=torch.int32))
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    out = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    out2 = torch.zeros_like(out)
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        k = (1.5 * torch.randn(L, B, Hkv, D)).bfloat16().cuda()
        v = (1.5 * torch.randn(L, B, Hkv, D)).bfloat16().cuda()
        if step == 3:
            k[0, 0, 0, :4] = torch.tensor([1e4, -1e4, 0.0, 3e-4]).bfloat16()      # saturation and underflow on the device
        lt.decode_step(fus.shape, q, k, v, fus.tables, fus.mask, fus.seq_lens, out, fus.ws)
        lt.kv_append(sep.shape, sep.mask, k, v, sep.seq_lens, sep.tables, ws=sep.ws)
        lt.hybrid_decode_attn(sep.shape, q, sep.tables, sep.mask, sep.seq_lens, out2, sep.ws)
        assert torch.equal(out, out2), step                                    # fused == append + attend, bit for bit
        for l in range(L):
            kc, kval = O.quantize_e4m3(f64(k[l]), scales[l, 0])
            vc, vval = O.quantize_e4m3(f64(v[l]), scales[l, 1])
            for b in range(B):
                replays[b].append(l, kval[b], vval[b])
                codes_hist[l][b] = np.concatenate([codes_hist[l][b], kc[b][:, None]], axis=1)
                mx, rel = attn_errors(f64(out[l, b]), replays[b].attend(l, f64(q[l, b])))
                assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (step, l, b, mx, rel)
    assert lt.check(fus.ws) == 0 and lt.check(sep.ws) == 0
    assert fus.seq_lens.cpu().tolist() == [n + steps for n in lens]
    for l in range(L):
        for st in (fus, sep):
            for b, n in enumerate(lens):
                for h in range(Hkv):
                    hist = codes_hist[l][b][h]                                  # [n + steps, D] codes
                    if mask[l]:
                        ek, _ = O.stream_cache_after(hist, S, R)
                        valid = O.ring_valid_slots(n + steps, S, R)
                        assert np.array_equal(st.k_stream[l][b, h, :valid].cpu().numpy(), ek[:valid])
                    else:
                        assert np.array_equal(st.k_full[l][b, h, :n + steps].cpu().numpy(), hist)


def test_fp8_shape_is_validated():
    sc = torch.full((2, 2), 0.02, dtype=torch.float32, device="cuda")
    ok = lt.Shape(2, 1, 8, 2, 128, 4, 12, 64, lt.LT_BF16, 0.0, kv_fp8=1, kv_scales=sc)
    assert lt.workspace_bytes(ok) > 0
    # scoring with 8-bit keys keeps a two-term copy of the tail queries in the workspace
    assert lt.workspace_bytes(ok, 64, 8) >= lt.workspace_bytes(ok) + 2 * (2 * 1 * 8 * 8) * 128
    for kw in (dict(kv_scales=None), dict(head_dim=64), dict(dtype=lt.LT_F32), dict(n_q_heads=66)):
        d = dict(ok.__dict__); d.update(kw)
        with pytest.raises(lt.LtError):
            lt.workspace_bytes(lt.Shape(**d))


@pytest.mark.parametrize("Hq,Hkv,T,n,S,R,per_row", [
    (8, 2, 64, 1500, 4, 60, 0),        # 256 query rows per kv head: both accumulators per tile; ragged last tile
    (5, 1, 16, 700, 4, 28, 0),         # 80 rows: one row block, tiles alternate between the accumulators
    (16, 2, 64, 900, 0, 100, 1),       # two query blocks per kv head; no sink; per-row window
    (8, 2, 32, 300, 4, 400, 0),        # the window covers every key: every score is 1
])
def test_fp8_keys_lazy_scores_match_eq1(Hq, Hkv, T, n, S, R, per_row):
    """Scoring from 8-bit keys (E4M3 MMAs on the stored bytes, q as two E4M3 terms) against Eq. 1 on the
    dequantised keys; the route with the log-sum-exp given must agree as well."""
    from tests.gpu_util import SCORE_ABS
    torch.manual_seed(41)
    g = np.random.default_rng(41)
    L, B, D = 2, 2, 128
    scales = g.uniform(0.015, 0.04, size=(L, 2)).astype(np.float32)
    sc = torch.from_numpy(scales).cuda().contiguous()
    shape = lt.Shape(L, B, Hq, Hkv, D, S, R, n, lt.LT_BF16, 0.0, recent_per_row=per_row, kv_fp8=1, kv_scales=sc)
    q_tail = torch.randn(L, B, Hq, T, D).bfloat16()
    q_tail[:, :, :, :, :3] *= 6.0                                              # a few large coordinates: the values of a row span several binades
    k8, kvals = [], []
    for l in range(L):
        hk = torch.randn(B, Hkv, n, D).bfloat16()
        hk[:, :, :max(S, 1)] += 0.3 * q_tail[l, :, ::Hq // Hkv].float().mean(2, keepdim=True).bfloat16()   # some mass on the first keys
        kc, kval = O.quantize_e4m3(f64(hk), scales[l, 0])
        k8.append(torch.from_numpy(kc).cuda()); kvals.append(kval)
    tables = lt.LayerTables(shape, k8, k8, None, None)
    ws = torch.empty(lt.workspace_bytes(shape, n, T), dtype=torch.uint8, device="cuda")
    lt.workspace_init(ws)
    scores = torch.full((L, B, Hq), float("nan"), device="cuda")
    lse_out = torch.full((L, B, Hq, T), float("nan"), device="cuda")
    lt.lazy_scores_with_lse(shape, q_tail.cuda(), tables, n, T, scores, lse_out, ws)
    ref = np.zeros((L, B, Hq)); lse = np.zeros((L, B, Hq, T))
    fn = O.lazy_scores_per_row_window if per_row else O.lazy_scores
    for l in range(L):
        for b in range(B):
            ref[l, b] = fn(f64(q_tail[l, b]), kvals[l][b], S, R)
            lse[l, b] = O.causal_lse(f64(q_tail[l, b]), kvals[l][b])
    assert lt.check(ws) == 0
    err = np.abs(f64(scores) - ref).max()
    assert err <= SCORE_ABS, err
    assert np.abs(f64(lse_out) - lse).max() <= 1e-3          # the denominators of the same pass, natural log
    if S + R >= n:
        assert np.abs(ref - 1.0).max() < 1e-12
    scores2 = torch.full((L, B, Hq), float("nan"), device="cuda")
    lt.lazy_scores_lse(shape, q_tail.cuda(), tables, torch.from_numpy(lse).float().cuda(), n, T, scores2, ws)
    assert lt.check(ws) == 0
    err2 = np.abs(f64(scores2) - ref).max()
    assert err2 <= SCORE_ABS, err2
    # one layer at a time writes the same bits into that layer's slice
    one = torch.full((L, B, Hq), float("nan"), device="cuda")
    for l in range(L):
        lt.lazy_scores(shape, q_tail.cuda(), tables, n, T, one, ws, layer_begin=l, layer_count=1)
    assert np.abs(f64(one) - ref).max() <= SCORE_ABS


def test_fp8_with_paged_full_caches():
    """Both options together: E4M3 pools behind a block table; 32-key tiles must not straddle pages."""
    torch.manual_seed(35)
    g = np.random.default_rng(35)
    L, B, Hq, Hkv, D, S, R, page, pps = 2, 2, 8, 2, 128, 4, 28, 128, 6
    cap = page * pps
    lens, steps = [600, 250], 12
    mask = np.array([0, 1], dtype=np.uint8)
    scales = g.uniform(0.015, 0.04, size=(L, 2)).astype(np.float32)
    n_pages = B * pps + 2
    table = torch.randperm(n_pages)[: B * pps].view(B, pps).to(torch.int32).cuda().contiguous()
    sc = torch.from_numpy(scales).cuda().contiguous()
    shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, lt.LT_BF16, 0.0, page_size=page, pages_per_seq=pps, n_pages=n_pages,
                     block_table=table, kv_fp8=1, kv_scales=sc)
    k_pool = [torch.zeros((n_pages, Hkv, page, D), dtype=torch.uint8, device="cuda") for _ in range(L)]
    v_pool = [torch.zeros((n_pages, Hkv, page, D), dtype=torch.uint8, device="cuda") for _ in range(L)]
    k_str = [torch.zeros((B, Hkv, S + R, D), dtype=torch.uint8, device="cuda") for _ in range(L)]
    v_str = [torch.zeros((B, Hkv, S + R, D), dtype=torch.uint8, device="cuda") for _ in range(L)]
    tables = lt.LayerTables(shape, k_pool, v_pool, k_str, v_str)
    ws = torch.empty(lt.workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    lt.workspace_init(ws)
    replays = [O.HybridReplay(mask, S, R) for _ in range(B)]
    tab = table.cpu()
    for l in range(L):
        hk = torch.randn(B, Hkv, cap, D).bfloat16(); hv = torch.randn(B, Hkv, cap, D).bfloat16()
        kc, kval = O.quantize_e4m3(f64(hk), scales[l, 0]); vc, vval = O.quantize_e4m3(f64(hv), scales[l, 1])
        for b in range(B):
            for p in range(pps):
                sl = slice(p * page, (p + 1) * page)
                k_pool[l][int(tab[b, p])] = torch.from_numpy(kc[b, :, sl]).cuda()
                v_pool[l][int(tab[b, p])] = torch.from_numpy(vc[b, :, sl]).cuda()
            replays[b].load_prompt(l, kval[b, :, :lens[b]], vval[b, :, :lens[b]])
    dmask = torch.from_numpy(mask).cuda()
    seq = torch.tensor(lens, dtype=torch.int32, device="cuda")
    lt.stream_init(shape, dmask, tables, seq, ws=ws)
    out = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda(); v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        lt.decode_step(shape, q, k, v, tables, dmask, seq, out, ws)
        for l in range(L):
            _, kval = O.quantize_e4m3(f64(k[l]), scales[l, 0]); _, vval = O.quantize_e4m3(f64(v[l]), scales[l, 1])
            for b in range(B):
                replays[b].append(l, kval[b], vval[b])
                mx, rel = attn_errors(f64(out[l, b]), replays[b].attend(l, f64(q[l, b])))
                assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (step, l, b, mx, rel)
    assert lt.check(ws) == 0 and seq.cpu().tolist() == [n + steps for n in lens]


def test_fp8_long_context_sampled_units():
    """Enough keys that a launch uses its longest (8192-key) chunks and several of them per unit;
    sampled (layer, batch row, kv head) units against the oracle on the dequantised values."""
    torch.manual_seed(37)
    g = np.random.default_rng(37)
    L, B, Hq, Hkv, D, S, R = 4, 4, 32, 8, 128, 4, 2044
    n0, steps = 40000, 2
    cap = n0 + steps
    mask = np.array([0, 1, 0, 1], dtype=np.uint8)
    scales = g.uniform(0.02, 0.04, size=(L, 2)).astype(np.float32)
    st = Fp8Stack(L, B, Hq, Hkv, S, R, cap, scales)
    table = torch.from_numpy(O.e4m3_values()).float().cuda()                 # code -> value, for the sampled read-back
    for l in range(L):
        st.k_full[l].copy_(torch.randint(0, 0x7F, st.k_full[l].shape, dtype=torch.uint8, device="cuda")
                           | (torch.randint(0, 2, st.k_full[l].shape, dtype=torch.uint8, device="cuda") << 7))
        st.v_full[l].copy_(torch.randint(0, 0x7F, st.v_full[l].shape, dtype=torch.uint8, device="cuda")
                           | (torch.randint(0, 2, st.v_full[l].shape, dtype=torch.uint8, device="cuda") << 7))
        st.k_full[l].clamp_(max=0xFE)                                        # keep the NaN codes out
        st.k_full[l][st.k_full[l] == 0x7F] = 0x7E
        st.v_full[l].clamp_(max=0xFE)
        st.v_full[l][st.v_full[l] == 0x7F] = 0x7E
    st.mask.copy_(torch.from_numpy(mask)); st.seq_lens.fill_(n0)
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    out = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    new = []
    for step in range(steps):
        q = (0.05 * torch.randn(L, B, Hq, D)).bfloat16().cuda()             # codes are spread over E4M3's whole range: keep logits moderate
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda(); v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        new.append((k, v))
        lt.decode_step(st.shape, q, k, v, st.tables, st.mask, st.seq_lens, out, st.ws)
    assert lt.check(st.ws) == 0 and torch.isfinite(out).all()
    G = Hq // Hkv
    for l, b, h in [(0, 0, 0), (1, 3, 7), (2, 1, 4), (3, 2, 5)]:
        Kq = table[st.k_full[l][b, h, :n0].long()].double().cpu().numpy() * float(scales[l, 0])
        Vq = table[st.v_full[l][b, h, :n0].long()].double().cpu().numpy() * float(scales[l, 1])
        ka = np.stack([O.quantize_e4m3(f64(k_[l, b, h]), scales[l, 0])[1] for k_, _ in new])
        va = np.stack([O.quantize_e4m3(f64(v_[l, b, h]), scales[l, 1])[1] for _, v_ in new])
        K = np.concatenate([Kq, ka])[None]; V = np.concatenate([Vq, va])[None]
        qh = f64(q[l, b, h * G:(h + 1) * G])
        ref = O.streaming_attention(qh, K, V, S, R) if mask[l] else O.full_attention(qh, K, V)
        mx, rel = attn_errors(f64(out[l, b, h * G:(h + 1) * G]), ref)
        assert rel <= ATTN_REL_L2 and mx <= ATTN_MAX_ABS * max(1.0, float(np.abs(ref).max())), (l, b, h, mx, rel)


def test_fp8_keys_lazy_scores_with_paged_pools():
    """Scoring from E4M3 page pools behind a block table: a 128-key box of a tile never straddles a page."""
    from tests.gpu_util import SCORE_ABS
    torch.manual_seed(43)
    g = np.random.default_rng(43)
    L, B, Hq, Hkv, D, S, R, page, pps, T = 2, 2, 8, 2, 128, 4, 60, 128, 9, 64
    cap, n = page * pps, 1100
    scales = g.uniform(0.015, 0.04, size=(L, 2)).astype(np.float32)
    n_pages = B * pps + 3
    table = torch.randperm(n_pages)[: B * pps].view(B, pps).to(torch.int32).cuda().contiguous()
    shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, lt.LT_BF16, 0.0, page_size=page, pages_per_seq=pps, n_pages=n_pages,
                     block_table=table, kv_fp8=1, kv_scales=torch.from_numpy(scales).cuda().contiguous())
    pools = [torch.full((n_pages, Hkv, page, D), 0x7E, dtype=torch.uint8, device="cuda") for _ in range(L)]   # 448 where nothing is stored
    q_tail = torch.randn(L, B, Hq, T, D).bfloat16()
    kvals, tab = [], table.cpu()
    for l in range(L):
        hk = torch.randn(B, Hkv, n, D).bfloat16()
        kc, kval = O.quantize_e4m3(f64(hk), scales[l, 0])
        kvals.append(kval)
        for b in range(B):
            for p in range(pps):
                lo, hi = p * page, min((p + 1) * page, n)
                if lo < hi:
                    pools[l][int(tab[b, p]), :, : hi - lo] = torch.from_numpy(kc[b, :, lo:hi]).cuda()
    tables = lt.LayerTables(shape, pools, pools, None, None)
    ws = torch.empty(lt.workspace_bytes(shape, n, T), dtype=torch.uint8, device="cuda")
    lt.workspace_init(ws)
    scores = torch.full((L, B, Hq), float("nan"), device="cuda")
    lt.lazy_scores(shape, q_tail.cuda(), tables, n, T, scores, ws)
    assert lt.check(ws) == 0
    ref = np.stack([np.stack([O.lazy_scores(f64(q_tail[l, b]), kvals[l][b], S, R) for b in range(B)]) for l in range(L)])
    err = np.abs(f64(scores) - ref).max()
    assert err <= SCORE_ABS and 0.0 < ref.min() and ref.max() < 0.9, (err, ref.min(), ref.max())


def test_fp8_32k_stack_scoring_from_8bit_keys_sampled_units():
    """The benchmark stack's shape with its keys stored as E4M3 (torch's cast makes the input codes, one scale per
    layer): scores from the 8-bit keys against Eq. 1 on the dequantised keys of sampled (layer, batch row, kv head)
    units - every kv head, first and last batch row, planted and unplanted layers - and the planted layers recovered."""
    import gc
    from synth import CONFIGS, make_layer, planted_layers
    from tests.gpu_util import SCORE_ABS
    gc.collect(); torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 30 * 2**30:
        pytest.skip("needs ~15 GB of free device memory")
    cfg = CONFIGS["llama3_8b_32k"]
    L, B, Hq, Hkv, D, n, T, G = (cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_ctx,
                                 cfg.w_last, cfg.group)
    planted = planted_layers(cfg)
    scales = np.full((L, 2), 0.03, dtype=np.float32)                     # |k| up to 448 x 0.03 = 13 is representable
    shape = lt.Shape(L, B, Hq, Hkv, D, cfg.n_sink, cfg.n_recent, n, lt.LT_BF16, 0.0, kv_fp8=1,
                     kv_scales=torch.from_numpy(scales).cuda().contiguous())
    q_tail = torch.empty((L, B, Hq, T, D), dtype=torch.bfloat16, device="cuda")
    k8 = []
    for l in range(L):
        qt, K, V = make_layer(cfg, l, l in planted, "cuda", capacity=n)
        q_tail[l].copy_(qt)
        k8.append((K.float() / 0.03).to(torch.float8_e4m3fn).view(torch.uint8).contiguous())
        del qt, K, V
    tables = lt.LayerTables(shape, k8, k8, None, None)
    ws = torch.empty(lt.workspace_bytes(shape, n, T), dtype=torch.uint8, device="cuda")
    lt.workspace_init(ws)
    scores = torch.zeros((L, B, Hq), dtype=torch.float32, device="cuda")
    lt.lazy_scores(shape, q_tail, tables, n, T, scores, ws)
    assert lt.check(ws) == 0
    sc = f64(scores)
    assert np.isfinite(sc).all() and sc.min() >= 0 and sc.max() <= 1 + 1e-6
    table = O.e4m3_values()                                              # code -> value, the oracle's own table
    unplanted = [l for l in range(L) if l not in planted]
    units = [(planted[0], 0, 0), (unplanted[0], B - 1, 1), (planted[-1], B - 1, 2), (unplanted[-1], 0, 3),
             (planted[len(planted) // 2], B // 2, 4), (unplanted[len(unplanted) // 2], 1, 5),
             (planted[1], B - 1, 6), (unplanted[1], 0, 7)]
    assert {u[2] for u in units} == set(range(Hkv))
    for l, b, h in units:
        Kd = table[k8[l][b, h].cpu().numpy()] * float(scales[l, 0])        # [n, D] dequantised keys of the unit
        ref = O.lazy_scores(f64(q_tail[l, b, h * G:(h + 1) * G]), Kd[None], cfg.n_sink, cfg.n_recent)
        assert np.max(np.abs(sc[l, b, h * G:(h + 1) * G] - ref)) <= SCORE_ABS, (l, b, h)
    mask = torch.zeros(L, dtype=torch.uint8, device="cuda")
    lt.select_lazy(scores, L, B, Hq, cfg.n_lazy, mask)
    assert sorted(np.nonzero(mask.cpu().numpy())[0].tolist()) == planted
    assert np.array_equal(mask.cpu().numpy(), O.select_lazy(sc, cfg.n_lazy)[0])
