"""GPU parity with paged full caches (block tables): every call that touches a
full cache follows block_table, and gives what the contiguous layout gives.
Paging is addressing only, so the oracle is the same logical-history oracle."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, SCORE_ABS, Stack, attn_errors, bits, f64, lt_dtype

pytestmark = pytest.mark.gpu


class PagedStack:
    """Page pools [n_pages][Hkv][page][D] per layer behind a shuffled block table;
    pages that no sequence owns hold NaN."""

    def __init__(self, L, B, Hq, Hkv, D, S, R, page, pages_per_seq, dtype, seed, spare=3, **shape_kw):
        g = torch.Generator().manual_seed(seed)
        self.n_pages = B * pages_per_seq + spare
        perm = torch.randperm(self.n_pages, generator=g)[: B * pages_per_seq]
        self.table = perm.view(B, pages_per_seq).to(torch.int32).cuda().contiguous()
        cap = page * pages_per_seq
        self.shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, lt_dtype(dtype), 0.0, page_size=page,
                              pages_per_seq=pages_per_seq, n_pages=self.n_pages, block_table=self.table, **shape_kw)
        self.page, self.dtype = page, dtype
        mk = lambda: [torch.full((self.n_pages, Hkv, page, D), float("nan"), dtype=dtype, device="cuda") for _ in range(L)]
        self.k_pool, self.v_pool = mk(), mk()
        self.k_stream = [torch.zeros((B, Hkv, S + R, D), dtype=dtype, device="cuda") for _ in range(L)]
        self.v_stream = [torch.zeros((B, Hkv, S + R, D), dtype=dtype, device="cuda") for _ in range(L)]
        self.tables = lt.LayerTables(self.shape, self.k_pool, self.v_pool, self.k_stream, self.v_stream)
        self.ws = torch.empty(lt.workspace_bytes(self.shape, cap, 64), dtype=torch.uint8, device="cuda")
        lt.workspace_init(self.ws)
        self.seq_lens = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.mask = torch.zeros(L, dtype=torch.uint8, device="cuda")

    def scatter(self, l, k_logical, v_logical):
        """Logical [B][Hkv][cap][D] -> pages."""
        B = k_logical.shape[0]
        tab = self.table.cpu()
        for b in range(B):
            for p in range(tab.shape[1]):
                sl = slice(p * self.page, (p + 1) * self.page)
                self.k_pool[l][int(tab[b, p])] = k_logical[b, :, sl].cuda()
                self.v_pool[l][int(tab[b, p])] = v_logical[b, :, sl].cuda()

    def gather(self, pool):
        """Pages -> logical [B][Hkv][cap][D]."""
        tab = self.table.long()
        x = pool[tab]                                   # [B, pps, Hkv, page, D]
        return x.permute(0, 2, 1, 3, 4).reshape(tab.shape[0], pool.shape[1], -1, pool.shape[3])


CASES = [
    # dtype, D, Hq, Hkv, S, R, page, pages_per_seq, lens, T
    (torch.bfloat16, 128, 8, 2, 4, 60, 128, 5, [300, 127, 128, 511], 32),      # tensor-core paths, page boundaries
    (torch.bfloat16, 128, 5, 1, 0, 16, 256, 9, [2040, 255], 8),                # G=5, several chunks over several pages
    (torch.float32, 64, 4, 2, 4, 28, 128, 3, [200, 40], 16),                   # CUDA-core paths
    (torch.bfloat16, 64, 8, 2, 4, 60, 128, 20, [2300, 129, 2048], 16),         # head_dim 64: 32-key tiles over page boundaries
    (torch.bfloat16, 128, 32, 2, 4, 60, 128, 20, [2300, 129, 2048], 8),        # G=16: warp pairs, 32-key tiles over page boundaries
    (torch.bfloat16, 64, 12, 1, 4, 28, 128, 5, [300, 511], 8),                 # head_dim 64, G=12: warp pairs
]


@pytest.mark.parametrize("dtype,D,Hq,Hkv,S,R,page,pps,lens,T", CASES)
def test_paged_path_equals_contiguous_path_and_oracle(dtype, D, Hq, Hkv, S, R, page, pps, lens, T):
    torch.manual_seed(23)
    L, B = 3, len(lens)
    cap = page * pps
    steps = 6
    mask = [0, 1, 0]
    pg = PagedStack(L, B, Hq, Hkv, D, S, R, page, pps, dtype, seed=24)
    ct = Stack(L, B, Hq, Hkv, D, S, R, cap, dtype, n_ctx_max=cap, w_last_max=64)
    hk = [torch.randn(B, Hkv, cap, D).to(dtype) for _ in range(L)]
    hv = [torch.randn(B, Hkv, cap, D).to(dtype) for _ in range(L)]
    for l in range(L):
        pg.scatter(l, hk[l], hv[l]); ct.k_full[l].copy_(hk[l]); ct.v_full[l].copy_(hv[l])
    # ---- scoring, both routes (all rows at the shortest common prompt length) ----
    n_ctx = min(lens)
    if n_ctx >= T:
        q_tail = (1.3 * torch.randn(L, B, Hq, T, D)).to(dtype).cuda()
        ref = np.array([[O.lazy_scores(f64(q_tail[l, b]), f64(hk[l][b, :, :n_ctx]), S, R) for b in range(B)]
                        for l in range(L)])
        got = torch.zeros((L, B, Hq), dtype=torch.float32, device="cuda")
        lt.lazy_scores(pg.shape, q_tail, pg.tables, n_ctx, T, got, pg.ws)
        assert np.max(np.abs(f64(got) - ref)) <= SCORE_ABS
        lse = torch.from_numpy(np.array([[O.causal_lse(f64(q_tail[l, b]), f64(hk[l][b, :, :n_ctx]))
                                          for b in range(B)] for l in range(L)])).float().cuda().contiguous()
        got2 = torch.zeros_like(got)
        lt.lazy_scores_lse(pg.shape, q_tail, pg.tables, lse, n_ctx, T, got2, pg.ws)
        assert np.max(np.abs(f64(got2) - ref)) <= SCORE_ABS
    # ---- compaction ----
    for st in (pg, ct):
        st.mask.copy_(torch.tensor(mask, dtype=torch.uint8)); st.seq_lens.copy_(torch.tensor(lens, dtype=torch.int32))
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    for l in range(L):
        assert torch.equal(pg.k_stream[l], ct.k_stream[l]) and torch.equal(pg.v_stream[l], ct.v_stream[l])
    # ---- decode steps: fused on the paged stack, append + attend on the contiguous one ----
    replays = []
    for b in range(B):
        rp = O.HybridReplay(mask, S, R)
        for l in range(L):
            rp.load_prompt(l, f64(hk[l][b, :, :lens[b]]), f64(hv[l][b, :, :lens[b]]))
        replays.append(rp)
    out = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    out2 = torch.zeros_like(out)
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).to(dtype).cuda()
        k = torch.randn(L, B, Hkv, D).to(dtype).cuda()
        v = torch.randn(L, B, Hkv, D).to(dtype).cuda()
        if step % 2 == 0:
            lt.decode_step(pg.shape, q, k, v, pg.tables, pg.mask, pg.seq_lens, out, pg.ws)
        else:                                                   # the separate calls follow the table too
            lt.kv_append(pg.shape, pg.mask, k, v, pg.seq_lens, pg.tables, ws=pg.ws)
            lt.hybrid_decode_attn(pg.shape, q, pg.tables, pg.mask, pg.seq_lens, out, pg.ws)
        ct.append(k, v)
        lt.hybrid_decode_attn(ct.shape, q, ct.tables, ct.mask, ct.seq_lens, out2, ct.ws)
        assert float((out - out2).abs().max()) <= 2e-3           # same arithmetic up to chunk boundaries
        for l in range(L):
            for b in range(B):
                replays[b].append(l, f64(k[l, b]), f64(v[l, b]))
                mx, rel = attn_errors(f64(out[l, b]), replays[b].attend(l, f64(q[l, b])))
                assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (step, l, b, mx, rel)
    assert lt.check(pg.ws) == 0 and torch.equal(pg.seq_lens, ct.seq_lens)
    for l in range(L):
        kl, vl = pg.gather(pg.k_pool[l]), pg.gather(pg.v_pool[l])
        for b in range(B):
            n = lens[b] + steps
            assert np.array_equal(bits(kl[b, :, :n]), bits(ct.k_full[l][b, :, :n]))
            assert np.array_equal(bits(vl[b, :, :n]), bits(ct.v_full[l][b, :, :n]))
        assert torch.equal(pg.k_stream[l], ct.k_stream[l])
        # pages that no sequence owns were never written
        owned = set(pg.table.flatten().tolist())
        for pidx in range(pg.n_pages):
            if pidx not in owned:
                assert bool(torch.isnan(pg.k_pool[l][pidx].float()).all())


def test_paging_arguments_are_validated_on_the_host():
    tab = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
    ok = lt.Shape(1, 2, 4, 1, 128, 4, 12, 512, page_size=128, pages_per_seq=4, n_pages=9, block_table=tab)
    assert lt.workspace_bytes(ok) > 0
    for kw in (dict(page_size=100), dict(full_capacity=500), dict(block_table=None), dict(n_pages=0)):
        d = dict(ok.__dict__); d.update(kw)
        with pytest.raises(lt.LtError):
            lt.workspace_bytes(lt.Shape(**d))
