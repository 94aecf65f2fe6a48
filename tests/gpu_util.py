"""Helpers shared by the GPU parity tests: device allocation through torch,
bit-exact copies back to the host, and the error metrics of the parity bar."""
import numpy as np
import torch

import paper_2410_13846_b200 as lt


def f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a device/host tensor's values to float64 numpy."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit patterns (int16 for bf16, int32 for fp32) on the host."""
    t = t.detach().to("cpu").contiguous()
    return t.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).numpy()


def lt_dtype(t):
    return lt.LT_F32 if t == torch.float32 else lt.LT_BF16


class Stack:
    """Device state of one attention stack: full and stream caches for every
    layer, tables, workspace, seq_lens, mask."""

    def __init__(self, L, B, Hq, Hkv, D, S, R, cap, dtype=torch.bfloat16, scale=0.0, n_ctx_max=0, w_last_max=0,
                 device="cuda"):
        self.shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, lt_dtype(dtype), scale)
        self.dtype, self.device = dtype, device
        self.k_full = [torch.zeros((B, Hkv, cap, D), dtype=dtype, device=device) for _ in range(L)]
        self.v_full = [torch.zeros((B, Hkv, cap, D), dtype=dtype, device=device) for _ in range(L)]
        self.k_stream = [torch.zeros((B, Hkv, S + R, D), dtype=dtype, device=device) for _ in range(L)]
        self.v_stream = [torch.zeros((B, Hkv, S + R, D), dtype=dtype, device=device) for _ in range(L)]
        self.tables = lt.LayerTables(self.shape, self.k_full, self.v_full, self.k_stream, self.v_stream)
        nbytes = lt.workspace_bytes(self.shape, n_ctx_max, w_last_max)
        self.ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
        assert self.ws.data_ptr() % 256 == 0
        lt.workspace_init(self.ws)
        self.seq_lens = torch.zeros(B, dtype=torch.int32, device=device)
        self.mask = torch.zeros(L, dtype=torch.uint8, device=device)

    def set_mask(self, mask):
        self.mask.copy_(torch.as_tensor(np.asarray(mask, dtype=np.uint8)))

    def set_seq_lens(self, lens):
        self.seq_lens.copy_(torch.as_tensor(np.asarray(lens, dtype=np.int32)))

    def attend(self, q, out_dtype=torch.float32, hint=0, **kw):
        s = self.shape
        out = torch.full((s.n_layers, s.batch, s.n_q_heads, s.head_dim), float("nan"), dtype=out_dtype,
                         device=self.device)
        lt.hybrid_decode_attn(s, q, self.tables, self.mask, self.seq_lens, out, self.ws, max_seq_len_hint=hint, **kw)
        return out

    def append(self, k_new, v_new, **kw):
        lt.kv_append(self.shape, self.mask, k_new, v_new, self.seq_lens, self.tables, ws=self.ws, **kw)


def attn_errors(got: np.ndarray, ref: np.ndarray):
    """(max abs error, relative L2 error) over the whole array."""
    diff = got - ref
    return float(np.max(np.abs(diff))), float(np.linalg.norm(diff) / max(np.linalg.norm(ref), 1e-300))


# the parity bar for attention outputs on bf16 inputs with fp32 accumulation
ATTN_MAX_ABS = 1e-2
ATTN_REL_L2 = 2e-3
SCORE_ABS = 1e-3


def build_stack(cfg, steps=None):
    """Device state of a synth workload: prompt K/V in the full caches of every
    layer, tail queries, seq_lens at the prompt length.  Returns (stack, q_tail,
    planted layers)."""
    from synth import make_layer, planted_layers, torch_dtype
    dt = torch_dtype(cfg)
    cap = cfg.n_ctx + (cfg.steps if steps is None else steps)
    st = Stack(cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_sink, cfg.n_recent, cap,
               dt, 0.0, n_ctx_max=cfg.n_ctx, w_last_max=cfg.w_last)
    planted = planted_layers(cfg)
    q_tail = torch.empty((cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.w_last, cfg.head_dim), dtype=dt, device="cuda")
    for l in range(cfg.n_layers):
        qt, K, V = make_layer(cfg, l, l in planted, "cuda", capacity=cap)
        q_tail[l].copy_(qt); st.k_full[l].copy_(K); st.v_full[l].copy_(V)
        del qt, K, V
    st.set_seq_lens([cfg.n_ctx] * cfg.batch)
    return st, q_tail, planted
