"""GPU parity on seeded random combinations of the options: group sizes across every kernel branch (one, two
or four warps per tile, CUDA-core passes), both head dimensions, fp32, ragged and empty rows, per-prompt masks,
paged full caches, tiny windows.  Each draw runs compaction and a few fused decode steps and is compared with
the oracle's replay on the logical history (O1 / O2 / O5), every (layer, batch row) of every step."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, Stack, attn_errors, bits, f64
from tests.test_gpu_paged import PagedStack

pytestmark = pytest.mark.gpu

GROUPS = [1, 2, 3, 4, 5, 7, 8, 9, 12, 16, 17, 20, 24, 31, 32, 33, 40]


def _draw(seed):
    g = np.random.default_rng(1000 + seed)
    cfg = dict(
        dtype=torch.float32 if g.random() < 0.2 else torch.bfloat16,
        D=int(g.choice([64, 128])),
        Hkv=int(g.choice([1, 2, 3])),
        G=int(GROUPS[seed % len(GROUPS)]),                 # every group size is drawn at least once
        S=int(g.choice([0, 1, 4, 7])),
        R=int(g.choice([1, 5, 16, 60, 300])),
        B=int(g.choice([1, 2, 3])),
        per_seq=bool(g.random() < 0.3),
        paged=bool(g.random() < 0.4),
        page=int(g.choice([128, 256])),
        steps=3,
    )
    cfg["lens"] = [int(x) for x in g.choice([0, 1, 2, 31, 127, 128, 129, 600, 2047, 2048, 2049, 2600], size=cfg["B"])]
    L = 3
    cfg["mask"] = (g.random((cfg["B"], L)) < 0.5).astype(np.uint8) if cfg["per_seq"] else \
        np.tile((g.random(L) < 0.5).astype(np.uint8), (cfg["B"], 1))
    return cfg


@pytest.mark.parametrize("seed", range(34))
def test_random_option_combinations_against_the_oracle(seed):
    c = _draw(seed)
    torch.manual_seed(2000 + seed)
    L, B, D, Hkv, G, S, R, steps = 3, c["B"], c["D"], c["Hkv"], c["G"], c["S"], c["R"], c["steps"]
    Hq, dtype, lens = Hkv * G, c["dtype"], c["lens"]
    need = max(lens) + steps
    if c["paged"]:
        pps = -(-need // c["page"])
        st = PagedStack(L, B, Hq, Hkv, D, S, R, c["page"], pps, dtype, seed=seed, per_sequence_mask=int(c["per_seq"]))
        cap = c["page"] * pps
    else:
        cap = need + 2
        st = Stack(L, B, Hq, Hkv, D, S, R, cap, dtype)
        if c["per_seq"]:
            st.shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, st.shape.dtype, 0.0, per_sequence_mask=1)
    hk = [torch.randn(B, Hkv, cap, D).to(dtype) for _ in range(L)]
    hv = [torch.randn(B, Hkv, cap, D).to(dtype) for _ in range(L)]
    for l in range(L):
        if c["paged"]:
            st.scatter(l, hk[l], hv[l])
        else:
            st.k_full[l].copy_(hk[l]); st.v_full[l].copy_(hv[l])
    mask_dev = torch.from_numpy(c["mask"] if c["per_seq"] else c["mask"][0]).cuda().contiguous()
    seq = torch.tensor(lens, dtype=torch.int32, device="cuda")
    lt.stream_init(st.shape, mask_dev, st.tables, seq, ws=st.ws)
    replays = []
    for b in range(B):
        rp = O.HybridReplay(c["mask"][b], S, R)
        for l in range(L):
            rp.load_prompt(l, f64(hk[l][b, :, :lens[b]]), f64(hv[l][b, :, :lens[b]]))
        replays.append(rp)
    out = torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    k_hist = [[[bits(hk[l][b, :, :lens[b]])] for b in range(B)] for l in range(L)]
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).to(dtype).cuda()
        k = torch.randn(L, B, Hkv, D).to(dtype).cuda()
        v = torch.randn(L, B, Hkv, D).to(dtype).cuda()
        lt.decode_step(st.shape, q, k, v, st.tables, mask_dev, seq, out, st.ws)
        for l in range(L):
            for b in range(B):
                replays[b].append(l, f64(k[l, b]), f64(v[l, b]))
                mx, rel = attn_errors(f64(out[l, b]), replays[b].attend(l, f64(q[l, b])))
                assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (c, step, l, b, mx, rel)
                k_hist[l][b].append(bits(k[l, b])[:, None])
    assert lt.check(st.ws) == 0 and seq.cpu().tolist() == [n + steps for n in lens]
    # the rings of the lazy layers, bit for bit (O5)
    for l in range(L):
        for b in range(B):
            if c["mask"][b, l]:
                hist = np.concatenate(k_hist[l][b], axis=1)            # [Hkv, n, D] bit patterns
                for h in range(Hkv):
                    ek, valid = O.stream_cache_after(hist[h], S, R)
                    assert np.array_equal(bits(st.k_stream[l][b, h, :valid]), ek[:valid]), (c, l, b, h)


@pytest.mark.parametrize("seed", range(24))
def test_random_scoring_combinations_against_eq1(seed):
    """Eq. 1 through both routes (full denominator; log-sum-exp given) on seeded random shapes: group sizes, tail
    lengths from one query to several row blocks, windows smaller and larger than the prompt, both readings of
    X_recent, paged caches, and both scoring kernels."""
    from tests.gpu_util import SCORE_ABS
    g = np.random.default_rng(3000 + seed)
    torch.manual_seed(4000 + seed)
    dtype = torch.float32 if g.random() < 0.2 else torch.bfloat16
    D = int(g.choice([64, 128]))
    Hkv = int(g.choice([1, 2]))
    G = int(g.choice([1, 2, 4, 5, 8, 16]))
    T = int(g.choice([1, 5, 16, 64]))
    n = int(g.choice([T, T + 1, 130, 257, 700, 1500, 2600]))
    n = max(n, T)
    S = int(g.choice([0, 1, 4]))
    R = int(g.choice([1, 16, 60, 300, 4000]))
    per_row = int(g.random() < 0.3)
    paged = bool(g.random() < 0.4) and dtype == torch.bfloat16
    L, B, Hq = 2, 2, Hkv * G
    if paged:
        page = 128
        pps = -(-n // page)
        st = PagedStack(L, B, Hq, Hkv, D, S, R, page, pps, dtype, seed=seed, recent_per_row=per_row)
        cap = page * pps
    else:
        cap = n
        st = Stack(L, B, Hq, Hkv, D, S, R, cap, dtype, n_ctx_max=n, w_last_max=T)
        st.shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, st.shape.dtype, 0.0, recent_per_row=per_row)
    hk = [torch.randn(B, Hkv, cap, D).to(dtype) for _ in range(L)]
    for l in range(L):
        if paged:
            st.scatter(l, hk[l], hk[l])
        else:
            st.k_full[l].copy_(hk[l])
    q_tail = (1.2 * torch.randn(L, B, Hq, T, D)).to(dtype)
    fn = O.lazy_scores_per_row_window if per_row else O.lazy_scores
    ref = np.zeros((L, B, Hq)); lse = np.zeros((L, B, Hq, T))
    for l in range(L):
        for b in range(B):
            ref[l, b] = fn(f64(q_tail[l, b]), f64(hk[l][b, :, :n]), S, R)
            lse[l, b] = O.causal_lse(f64(q_tail[l, b]), f64(hk[l][b, :, :n]))
    ws = torch.empty(lt.workspace_bytes(st.shape, n, T), dtype=torch.uint8, device="cuda")
    lt.workspace_init(ws)
    a = torch.full((L, B, Hq), float("nan"), device="cuda")
    b2 = torch.full((L, B, Hq), float("nan"), device="cuda")
    lse_out = torch.full((L, B, Hq, T), float("nan"), device="cuda")
    lt.lazy_scores_with_lse(st.shape, q_tail.cuda(), st.tables, n, T, a, lse_out, ws)
    lt.lazy_scores_lse(st.shape, q_tail.cuda(), st.tables, torch.from_numpy(lse).float().cuda(), n, T, b2, ws)
    assert lt.check(ws) == 0
    what = (seed, dtype, D, Hkv, G, T, n, S, R, per_row, paged)
    assert np.max(np.abs(f64(a) - ref)) <= SCORE_ABS, what
    assert np.max(np.abs(f64(b2) - ref)) <= SCORE_ABS, what
    assert np.max(np.abs(f64(lse_out) - lse)) <= 2e-4, what
