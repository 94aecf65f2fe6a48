#!/usr/bin/env python
"""Benchmark of the hybrid decode-attention path on the Llama-3-8B-shaped 32K
stack (32 layers, 32 q / 8 kv heads, head_dim 128, bf16, batch 8, context 32768,
sink 4 + window 2044, 16 lazy layers, 128 decode steps).

One "step" of this benchmark is one whole pass of the hot path over one batch:
lazy scores over the last 64 prompt queries -> device top-k -> compaction of the
lazy layers -> 128 x (one fused launch: KV append + hybrid decode attention over
all 32 layers + seq_lens advance).
`value` = decode tokens of all ranks / time of the timed passes.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
  python bench.py --workload {llama2_7b_4k,llama31_8b_128k,qwq32b_longgen}   # one of the other workloads alone

N > 1 (under torch.distributed.run) runs one independent replica per GPU: the
path has no exchange step, so there is no data-path collective.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

WORKLOAD = "llama3_8b_32k"
METRIC = "hybrid decode-attn tokens/s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes of one decode-kernel launch as a ratio to the algorithmic bytes of that launch, from the
# committed DRAM-byte capture of the 4-layer small case (the counters are not read during a timed run, so
# the line's traffic figure is this constant ratio times the algorithmic bytes, and is labelled as such).
NCU_TRAFFIC_RATIO = 1.004


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def _tensor_peak():
    """Sustained dense bf16 TFLOP/s measured on this machine (fallback: an earlier measurement)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["bf16_tflops_sustained"])
    except Exception:
        return 1400.0


def _dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init_replicas(world: int, backend: str = "nccl", device=None):
    """Process group of the replicas (None for a single process).  The path has
    no exchange step: the group is used for the barrier around the timed region
    and for the max-over-ranks of the measured time, never for data."""
    if world <= 1:
        return None
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group(backend)
    return dist


def max_over_ranks(x: float, dist, device=None) -> float:
    """Slowest rank's time: every replica must have finished its steps."""
    if dist is None:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, tokens_per_rank: int, ms: float) -> float:
    """tokens/s of all replicas together over the slowest rank's time."""
    return world * tokens_per_rank / (ms * 1e-3)


# ----------------------------------------------------------------------------
# clocks sampling during the timed region
# ----------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "power_w": None}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, pw, reasons, mx = [], [], set(), None
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx = float(f[2])
                except ValueError:
                    continue
                try:
                    pw.append(float(f[3]))
                except ValueError:
                    pw.append(float("nan"))
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            # samples under load: drop the idle ones at the edges
            load = [x for x in sm if x > 0.5 * max(sm)]
            out.update(sm_mhz=float(np.median(load)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
            pw_load = [p for p, x in zip(pw, sm) if x > 0.5 * max(sm) and p == p]
            if pw_load:
                out["power_w"] = float(np.median(pw_load))      # board power under load (the cap is 1000 W)
        return out


# ----------------------------------------------------------------------------
# workload
# ----------------------------------------------------------------------------
def algorithmic_bytes_decode(cfg, n, n_lazy):
    """Bytes one decode step must move with every row at length n (after the
    append): K and V of every cached token once, plus q, out, k_new, v_new."""
    e = 2 if cfg.dtype == "bf16" else 4
    row = 2 * cfg.n_kv_heads * cfg.head_dim * e
    C = cfg.n_sink + cfg.n_recent
    kv = (cfg.n_layers - n_lazy) * cfg.batch * n * row + n_lazy * cfg.batch * min(n, C) * row
    small = cfg.n_layers * cfg.batch * cfg.head_dim * (2 * cfg.n_q_heads * e + 2 * cfg.n_kv_heads * e)
    return kv + small


class Workload:
    def __init__(self, cfg, device):
        import paper_2410_13846_b200 as lt
        from synth import make_layer, planted_layers, torch_dtype
        self.lt, self.cfg, self.device = lt, cfg, device
        dt = torch_dtype(cfg)
        L, B, Hq, Hkv, D = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        cap = cfg.n_ctx + cfg.steps
        self.shape = lt.Shape(L, B, Hq, Hkv, D, cfg.n_sink, cfg.n_recent, cap,
                              lt.LT_F32 if dt == torch.float32 else lt.LT_BF16)
        self.planted = planted_layers(cfg)
        C = cfg.n_sink + cfg.n_recent
        self.k_full, self.v_full = [], []
        self.q_tail = torch.empty((L, B, Hq, cfg.w_last, D), dtype=dt, device=device)
        for l in range(L):
            qt, K, V = make_layer(cfg, l, l in self.planted, device, capacity=cap)
            self.q_tail[l].copy_(qt); self.k_full.append(K); self.v_full.append(V)
        self.k_stream = [torch.zeros((B, Hkv, C, D), dtype=dt, device=device) for _ in range(L)]
        self.v_stream = [torch.zeros((B, Hkv, C, D), dtype=dt, device=device) for _ in range(L)]
        self.tables = lt.LayerTables(self.shape, self.k_full, self.v_full, self.k_stream, self.v_stream)
        self.ws = torch.empty(lt.workspace_bytes(self.shape, cfg.n_ctx, cfg.w_last), dtype=torch.uint8, device=device)
        lt.workspace_init(self.ws)
        self.seq = torch.zeros(B, dtype=torch.int32, device=device)
        self.seq0 = torch.full((B,), cfg.n_ctx, dtype=torch.int32, device=device)
        self.mask = torch.zeros(L, dtype=torch.uint8, device=device)
        self.scores = torch.zeros((L, B, Hq), dtype=torch.float32, device=device)
        self.out = torch.zeros((L, B, Hq, D), dtype=dt, device=device)
        # a few rotating sets of per-step inputs (their content does not change the work)
        from synth import decode_inputs
        self.step_inputs = [decode_inputs(cfg, s, device) for s in range(4)]
        self.launches = 0

    # -- pieces ---------------------------------------------------------------
    def identify(self):
        lt, cfg = self.lt, self.cfg
        lt.lazy_scores(self.shape, self.q_tail, self.tables, cfg.n_ctx, cfg.w_last, self.scores, self.ws)
        lt.select_lazy(self.scores, cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_lazy, self.mask)
        self.seq.copy_(self.seq0)
        lt.stream_init(self.shape, self.mask, self.tables, self.seq, ws=self.ws)
        self.launches += 4

    def decode_step(self, i, ev=None):
        lt = self.lt
        q, k, v = self.step_inputs[i % len(self.step_inputs)]
        if ev is not None:
            ev[0].record()
        # append + attend + merge + seq_lens advance: one launch
        lt.decode_step(self.shape, q, k, v, self.tables, self.mask, self.seq, self.out, self.ws)
        if ev is not None:
            ev[1].record()
        self.launches += 1

    def prefill_lse(self):
        """Log-sum-exp of the tail rows' scaled causal logits, as a prefill's
        attention kernel returns it (an INPUT of lt_lazy_scores_lse; made here
        once with plain torch ops, outside every timed region)."""
        cfg = self.cfg
        L, B, Hq, Hkv, D, T, n = (cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.w_last,
                                  cfg.n_ctx)
        G = Hq // Hkv
        lse = torch.empty((L, B, Hq, T), dtype=torch.float32, device=self.device)
        j = torch.arange(n, device=self.device)
        vis = j[None, :] <= (n - T + torch.arange(T, device=self.device))[:, None]          # [T, n]
        for l in range(L):
            for b in range(B):
                q = self.q_tail[l, b].float().view(Hkv, G * T, D)
                k = self.k_full[l][b, :, :n].float()                                        # [Hkv, n, D]
                logits = torch.bmm(q, k.transpose(1, 2)).view(Hkv, G, T, n) / (D ** 0.5)
                logits = logits.masked_fill(~vis[None, None], float("-inf"))
                lse[l, b] = torch.logsumexp(logits, dim=-1).view(Hq, T)
        return lse

    def full_pass(self, events=None):
        self.identify()
        for i in range(self.cfg.steps):
            self.decode_step(i, None if events is None else events[i])


def _event_pairs(n):
    return [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]


def run_ours(args):
    rank, local_rank, world = _dist_env()
    if args.gpus != world:
        if world == 1 and args.gpus > 1:
            raise SystemExit("--gpus N > 1 must be launched with torch.distributed.run (one rank per GPU)")
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = init_replicas(world, "nccl", device)

    from paper_2410_13846_b200 import build
    build.build_library()
    from synth import CONFIGS
    cfg = CONFIGS[WORKLOAD]
    wl = Workload(cfg, device)
    K, W = args.steps, max(args.warmup, 3)
    B, T = cfg.batch, cfg.steps

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up --------------------------------------------------------------
    for _ in range(W):
        wl.full_pass()
    torch.cuda.synchronize()
    mask = wl.mask.cpu().numpy()
    assert sorted(np.nonzero(mask)[0].tolist()) == wl.planted, "planted layers not recovered"
    assert wl.lt.check(wl.ws) == 0

    # ---- timed region: K whole passes --------------------------------------------
    events = [_event_pairs(T) for _ in range(K)]
    e_id = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cvd = os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",")
    gpu_index = int(cvd[local_rank]) if local_rank < len(cvd) and cvd[local_rank].isdigit() else local_rank
    sampler = ClockSampler(gpu_index)
    wl.launches = 0
    barrier()
    sampler.start()
    t0.record()
    for k in range(K):
        e_id[k][0].record()
        wl.identify()
        e_id[k][1].record()
        for i in range(T):
            wl.decode_step(i, events[k][i])
    t1.record()
    barrier()
    clocks = sampler.stop()
    total_ms = t0.elapsed_time(t1)
    launches = wl.launches
    total_ms = max_over_ranks(total_ms, dist, device)
    attn_ms = np.array([[a.elapsed_time(b) for a, b in ev] for ev in events])          # [K, T]
    ident_ms = np.array([a.elapsed_time(b) for a, b in e_id])
    decode_ms_total = total_ms - float(ident_ms.sum())

    # ---- derived numbers ----------------------------------------------------------
    value = whole_job_value(world, B * T * K, total_ms)
    bytes_per_step = np.array([algorithmic_bytes_decode(cfg, cfg.n_ctx + i + 1, cfg.n_lazy) for i in range(T)])
    attn_gbs = float(bytes_per_step.sum() * K / (attn_ms.sum() * 1e-3) / 1e9)
    peak, peak_kind = _peaks()

    # ---- the same kernels under the all-full mask (analogue of the paper's ratio) ----
    wl.mask.zero_(); wl.seq.copy_(wl.seq0)
    nfull = 24
    evf = _event_pairs(nfull)
    for i in range(4):
        wl.decode_step(i)
    torch.cuda.synchronize()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for i in range(nfull):
        wl.decode_step(i, evf[i])
    f1.record()
    torch.cuda.synchronize()
    full_step_ms = f0.elapsed_time(f1) / nfull
    full_attn_ms = float(np.mean([a.elapsed_time(b) for a, b in evf]))
    full_bytes = float(np.mean([algorithmic_bytes_decode(cfg, cfg.n_ctx + 4 + i + 1, 0) for i in range(nfull)]))

    # ---- the deployed identification: denominator from the prefill, window block only ----
    lse = wl.prefill_lse()
    scores_lse = torch.zeros_like(wl.scores)
    mask_lse = torch.zeros_like(wl.mask)
    lt = wl.lt
    for _ in range(3):
        lt.lazy_scores_lse(wl.shape, wl.q_tail, wl.tables, lse, cfg.n_ctx, cfg.w_last, scores_lse, wl.ws)
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(10):
        lt.lazy_scores_lse(wl.shape, wl.q_tail, wl.tables, lse, cfg.n_ctx, cfg.w_last, scores_lse, wl.ws)
    g1.record()
    torch.cuda.synchronize()
    lse_ms = g0.elapsed_time(g1) / 10
    lt.select_lazy(scores_lse, cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_lazy, mask_lse)
    assert sorted(np.nonzero(mask_lse.cpu().numpy())[0].tolist()) == wl.planted, "LSE route: planted layers not recovered"
    lt.lazy_scores(wl.shape, wl.q_tail, wl.tables, cfg.n_ctx, cfg.w_last, wl.scores, wl.ws)
    routes_diff = float((wl.scores - scores_lse).abs().max())
    del lse

    # ---- the scoring kernel alone against its three roofs (HBM, tensor, MUFU) -------------
    n_it = 400                         # about 2.4 s: long enough for the 200 ms clock and power samples to see the loop alone
    s_sampler = ClockSampler(gpu_index)
    torch.cuda.synchronize()
    s_sampler.start()
    g0.record()
    for _ in range(n_it):
        lt.lazy_scores(wl.shape, wl.q_tail, wl.tables, cfg.n_ctx, cfg.w_last, wl.scores, wl.ws)
    g1.record()
    torch.cuda.synchronize()
    s_clk = s_sampler.stop()
    score_ms = g0.elapsed_time(g1) / n_it
    L_, B_, Hq_, Hkv_, D_, T_, n_ = (cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.w_last,
                                     cfg.n_ctx)
    k_bytes = L_ * B_ * Hkv_ * n_ * D_ * 2
    flops = 2.0 * T_ * Hq_ * n_ * D_ * L_ * B_
    exps = float(T_) * Hq_ * n_ * L_ * B_
    mhz = s_clk["sm_mhz"] or clocks["sm_mhz"] or 1965.0
    mufu_peak = 16 * 148 * mhz * 1e6                       # one ex2 per lane, 16 lanes per clock per SM, 148 SMs
    tf_peak = _tensor_peak()
    score_roofs = {"ms": score_ms, "sm_mhz": mhz, "power_w": s_clk.get("power_w"), "clock_reasons": s_clk.get("reasons"),
                   "hbm": {"achieved_gbs": k_bytes / (score_ms * 1e-3) / 1e9, "frac": k_bytes / (score_ms * 1e-3) / 1e9 / peak},
                   "tensor": {"achieved_tflops": flops / (score_ms * 1e-3) / 1e12, "peak_tflops": tf_peak,
                              "frac": flops / (score_ms * 1e-3) / 1e12 / tf_peak},
                   "mufu": {"achieved_gexp_s": exps / (score_ms * 1e-3) / 1e9, "peak_gexp_s": mufu_peak / 1e9,
                            "frac": exps / (score_ms * 1e-3) / mufu_peak,
                            "peak_how": "16 ex2 per clock per SM x 148 SMs x the SM clock sampled during this loop"}}

    # ---- end to end through the public API with host buffers ----------------------
    e2e = run_e2e(wl, passes=max(1, min(K, 2)))
    e2e["ms_per_pass"] = max_over_ranks(e2e["ms_per_pass"], dist, device)
    e2e_value = whole_job_value(world, B * T, e2e["ms_per_pass"])

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, wl)

    # ---- the same step with paged and with 8-bit caches (detail only; last, it reuses the caches) ----
    mask_hybrid = torch.zeros_like(wl.mask)
    mask_hybrid[torch.as_tensor(wl.planted, device=device)] = 1
    variants = run_variants(wl, mask_hybrid) if world == 1 else {}
    per_layer = run_per_layer_calls(wl, mask_hybrid, peak) if world == 1 else None
    per_layer_over = run_per_layer_calls(wl, mask_hybrid, peak, overlapped=True) if world == 1 else None
    other = {}
    if world == 1 and not args.no_other_configs:
        # the other paper-shaped workloads, one stack at a time (the benchmark stack is freed first)
        del wl
        import gc
        gc.collect(); torch.cuda.empty_cache()
        other = run_other_configs(device, peak, gpu_index)

    if rank == 0:
        hybrid_step_ms = decode_ms_total / (K * T)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "layers": cfg.n_layers, "q_heads": cfg.n_q_heads,
                       "kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim, "batch": B, "context": cfg.n_ctx,
                       "n_sink": cfg.n_sink, "n_recent": cfg.n_recent, "w_last": cfg.w_last, "n_lazy": cfg.n_lazy,
                       "decode_steps_per_pass": T,
                       "step": "scores+select+compaction+128x(fused append+attend)",
                       "l2": "inputs (17 GiB per decode step) exceed the 126 MB L2; no flush needed",
                       "parallelism": "replicas" if world > 1 else "single"},
            "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons", "power_w")},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                    "ms_per_step": e2e["ms_per_pass"]},
            "gpu_launches": launches,
            "roofline": {"bound": "hbm", "achieved": attn_gbs, "peak": peak, "unit": "GB/s", "frac": attn_gbs / peak,
                         "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": attn_gbs / NOMINAL_HBM_GBS,
                         "kernel": "lt_decode_step (persistent split-KV kernel: append + attend + merge), hybrid mask",
                         "algorithmic_bytes_per_launch": float(bytes_per_step.mean()),
                         "ms_per_launch": float(attn_ms.mean()),
                         "traffic": (float(bytes_per_step.mean()) * NCU_TRAFFIC_RATIO) if NCU_TRAFFIC_RATIO else None,
                         "traffic_how": "estimated: algorithmic bytes x the DRAM-bytes / algorithmic-bytes ratio of the "
                                        "committed small-case ncu capture (not re-measured in this run)"},
            "cpu_baseline": cpu,
            "detail": {
                "hybrid": {"step_ms": hybrid_step_ms, "attn_ms": float(attn_ms.mean()),
                           "decode_tokens_per_s": world * B / (hybrid_step_ms * 1e-3), "attn_gbs": attn_gbs},
                "all_full": {"step_ms": full_step_ms, "attn_ms": full_attn_ms,
                             "decode_tokens_per_s": world * B / (full_step_ms * 1e-3),
                             "attn_gbs": full_bytes / (full_attn_ms * 1e-3) / 1e9,
                             "frac_of_peak": full_bytes / (full_attn_ms * 1e-3) / 1e9 / peak},
                "hybrid_over_all_full": full_step_ms / hybrid_step_ms,
                "byte_ratio_ceiling": full_bytes / float(bytes_per_step.mean()),
                "lazy_score_ms": float(ident_ms.mean()),
                "lazy_score_lse_route_ms": lse_ms,
                "lazy_score_routes_max_abs_diff": routes_diff,
                "lazy_score_kernel_roofs": score_roofs,
                "variants": variants,
                "per_layer_calls": per_layer,
                "per_layer_calls_overlapped": per_layer_over,
                "other_configs": other,
                "paper_context": "paper reports up to 2.17x whole-model throughput vs full attention on A100 "
                                 "(Mistral-7B, 16K, max batch); other hardware, not the target",
            },
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_variants(wl, mask_hybrid):
    """The same decode step on the same stack shape with (a) paged full caches
    (128-token pages behind a shuffled block table) and (b) FP8 E4M3 caches with
    per-layer scales; also with head_dim 64, with a query group of 16 and with fp32 caches
    (the CUDA-core kernels).  Contents are random: the work does not depend on them.
    Reported in `detail`; the headline stays the contiguous bf16 stack."""
    cfg, lt, dev = wl.cfg, wl.lt, wl.device
    L, B, Hq, Hkv, D = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    C = cfg.n_sink + cfg.n_recent
    q, k, v = wl.step_inputs[0]
    out = torch.zeros_like(wl.out)
    res = {}

    def time_steps(shape, tables, ws, n0, steps=16):
        seq = torch.full((B,), n0, dtype=torch.int32, device=dev)
        for _ in range(3):
            lt.decode_step(shape, q, k, v, tables, mask_hybrid, seq, out, ws)
        torch.cuda.synchronize()
        seq.fill_(n0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            lt.decode_step(shape, q, k, v, tables, mask_hybrid, seq, out, ws)
        e1.record()
        torch.cuda.synchronize()
        assert lt.check(ws) == 0
        return e0.elapsed_time(e1) / steps

    n_mean = cfg.n_ctx + 8.5
    # (a) paged: the benchmark's own K/V tensors viewed as page pools (same bytes, other addressing)
    page = 128
    cap = wl.shape.full_capacity
    if cap % page == 0:
        pps = cap // page
        n_pages = B * pps
        table = torch.randperm(n_pages, device=dev)[: B * pps].view(B, pps).to(torch.int32).contiguous()
        shape = lt.Shape(L, B, Hq, Hkv, D, cfg.n_sink, cfg.n_recent, cap, lt.LT_BF16, page_size=page,
                         pages_per_seq=pps, n_pages=n_pages, block_table=table)
        pools_k = [t.view(n_pages, Hkv, page, D) for t in wl.k_full]
        pools_v = [t.view(n_pages, Hkv, page, D) for t in wl.v_full]
        tables = lt.LayerTables(shape, pools_k, pools_v, wl.k_stream, wl.v_stream)
        ms = time_steps(shape, tables, wl.ws, cfg.n_ctx)
        res["paged_128"] = {"step_ms": ms, "decode_tokens_per_s": B / (ms * 1e-3),
                            "gbs": algorithmic_bytes_decode(cfg, n_mean, cfg.n_lazy) / (ms * 1e-3) / 1e9}
    # (b) FP8 caches: byte tensors of the same geometry
    scales = torch.full((L, 2), 0.02, dtype=torch.float32, device=dev)
    shape8 = lt.Shape(L, B, Hq, Hkv, D, cfg.n_sink, cfg.n_recent, cap, lt.LT_BF16, kv_fp8=1, kv_scales=scales)
    mk = lambda n: [torch.randint(0, 120, (B, Hkv, n, D), dtype=torch.uint8, device=dev) for _ in range(L)]
    k8, v8, ks8, vs8 = mk(cap), mk(cap), mk(C), mk(C)
    tables8 = lt.LayerTables(shape8, k8, v8, ks8, vs8)
    ws8 = torch.empty(lt.workspace_bytes(shape8), dtype=torch.uint8, device=dev)
    lt.workspace_init(ws8)
    ms = time_steps(shape8, tables8, ws8, cfg.n_ctx)
    kv8 = algorithmic_bytes_decode(cfg, n_mean, cfg.n_lazy) / 2          # one byte per cached element
    res["fp8_caches"] = {"step_ms": ms, "decode_tokens_per_s": B / (ms * 1e-3), "gbs_of_8bit_bytes": kv8 / (ms * 1e-3) / 1e9}
    # ... and the lazy scores over the whole prompt read from the 8-bit keys (E4M3 MMAs on the stored bytes)
    del ws8
    T8 = cfg.w_last
    ws8 = torch.empty(lt.workspace_bytes(shape8, cfg.n_ctx, T8), dtype=torch.uint8, device=dev)
    lt.workspace_init(ws8)
    sc8 = torch.zeros((L, B, Hq), dtype=torch.float32, device=dev)
    for _ in range(2):
        lt.lazy_scores(shape8, wl.q_tail, tables8, cfg.n_ctx, T8, sc8, ws8)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(20):
        lt.lazy_scores(shape8, wl.q_tail, tables8, cfg.n_ctx, T8, sc8, ws8)
    e1.record()
    torch.cuda.synchronize()
    assert lt.check(ws8) == 0 and bool(torch.isfinite(sc8).all())
    res["fp8_caches"]["lazy_scores_ms"] = e0.elapsed_time(e1) / 20
    del k8, v8, ks8, vs8, ws8, tables8, sc8
    # (c) the same stack with head_dim 64 (bf16): half the bytes per token, 32-key tiles of 128-byte rows
    shape64 = lt.Shape(L, B, Hq, Hkv, 64, cfg.n_sink, cfg.n_recent, cap, lt.LT_BF16)
    mk64 = lambda n: [torch.randn((B, Hkv, n, 64), device=dev).bfloat16() for _ in range(L)]  # noqa: E731
    k64, v64, ks64, vs64 = mk64(cap), mk64(cap), mk64(C), mk64(C)
    tables64 = lt.LayerTables(shape64, k64, v64, ks64, vs64)
    ws64 = torch.empty(lt.workspace_bytes(shape64), dtype=torch.uint8, device=dev)
    lt.workspace_init(ws64)
    q64, kn64 = (torch.randn((L, B, h, 64), device=dev).bfloat16() for h in (Hq, Hkv))
    out64 = torch.zeros((L, B, Hq, 64), dtype=torch.bfloat16, device=dev)
    seq = torch.full((B,), cfg.n_ctx, dtype=torch.int32, device=dev)
    for _ in range(3):
        lt.decode_step(shape64, q64, kn64, kn64, tables64, mask_hybrid, seq, out64, ws64)
    torch.cuda.synchronize()
    seq.fill_(cfg.n_ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(16):
        lt.decode_step(shape64, q64, kn64, kn64, tables64, mask_hybrid, seq, out64, ws64)
    e1.record()
    torch.cuda.synchronize()
    assert lt.check(ws64) == 0
    ms = e0.elapsed_time(e1) / 16
    b64 = algorithmic_bytes_decode(cfg.scaled(head_dim=64), n_mean, cfg.n_lazy)
    res["head_dim_64"] = {"step_ms": ms, "decode_tokens_per_s": B / (ms * 1e-3), "gbs": b64 / (ms * 1e-3) / 1e9}
    # ... and its lazy scores over the whole prompt (Eq. 1): the tensor-core kernel with four 16-wide k-steps per tile
    T = cfg.w_last
    wsS = torch.empty(lt.workspace_bytes(shape64, cfg.n_ctx, T), dtype=torch.uint8, device=dev)
    lt.workspace_init(wsS)
    qt64 = torch.randn((L, B, Hq, T, 64), device=dev).bfloat16()
    sc64 = torch.zeros((L, B, Hq), dtype=torch.float32, device=dev)
    for _ in range(2):
        lt.lazy_scores(shape64, qt64, tables64, cfg.n_ctx, T, sc64, wsS)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(3):
        lt.lazy_scores(shape64, qt64, tables64, cfg.n_ctx, T, sc64, wsS)
    e1.record()
    torch.cuda.synchronize()
    assert lt.check(wsS) == 0
    ms = e0.elapsed_time(e1) / 3
    res["head_dim_64"]["lazy_scores_ms"] = ms
    res["head_dim_64"]["lazy_scores_tflops"] = 2.0 * L * B * Hq * T * cfg.n_ctx * 64 / (ms * 1e-3) / 1e12
    del k64, v64, ks64, vs64, ws64, wsS, qt64, tables64
    # (d) a query group of 16 (32 q / 2 kv heads): two warps share every tile and serve eight heads each
    cfg16 = cfg.scaled(n_kv_heads=2)
    shape16 = lt.Shape(L, B, Hq, 2, D, cfg.n_sink, cfg.n_recent, cap, lt.LT_BF16)
    mk16 = lambda n: [torch.randn((B, 2, n, D), device=dev).bfloat16() for _ in range(L)]  # noqa: E731
    k16, v16, ks16, vs16 = mk16(cap), mk16(cap), mk16(C), mk16(C)
    tables16 = lt.LayerTables(shape16, k16, v16, ks16, vs16)
    ws16 = torch.empty(lt.workspace_bytes(shape16), dtype=torch.uint8, device=dev)
    lt.workspace_init(ws16)
    kn16 = torch.randn((L, B, 2, D), device=dev).bfloat16()
    seq = torch.full((B,), cfg.n_ctx, dtype=torch.int32, device=dev)
    for _ in range(3):
        lt.decode_step(shape16, q, kn16, kn16, tables16, mask_hybrid, seq, out, ws16)
    torch.cuda.synchronize()
    seq.fill_(cfg.n_ctx)
    e0.record()
    for _ in range(16):
        lt.decode_step(shape16, q, kn16, kn16, tables16, mask_hybrid, seq, out, ws16)
    e1.record()
    torch.cuda.synchronize()
    assert lt.check(ws16) == 0
    ms = e0.elapsed_time(e1) / 16
    b16 = algorithmic_bytes_decode(cfg16, n_mean, cfg.n_lazy)
    res["group_16"] = {"step_ms": ms, "decode_tokens_per_s": B / (ms * 1e-3), "gbs": b16 / (ms * 1e-3) / 1e9}
    del k16, v16, ks16, vs16, ws16, tables16
    # ... and a group of 32 (64 q / 2 kv heads): the four warps share every tile and serve eight heads each
    cfg32g = cfg.scaled(n_q_heads=64, n_kv_heads=2)
    shape32g = lt.Shape(L, B, 64, 2, D, cfg.n_sink, cfg.n_recent, cap, lt.LT_BF16)
    k16, v16, ks16, vs16 = mk16(cap), mk16(cap), mk16(C), mk16(C)
    tables32g = lt.LayerTables(shape32g, k16, v16, ks16, vs16)
    ws32g = torch.empty(lt.workspace_bytes(shape32g), dtype=torch.uint8, device=dev)
    lt.workspace_init(ws32g)
    q32g = torch.randn((L, B, 64, D), device=dev).bfloat16()
    out32g = torch.zeros_like(q32g)
    seq = torch.full((B,), cfg.n_ctx, dtype=torch.int32, device=dev)
    for _ in range(3):
        lt.decode_step(shape32g, q32g, kn16, kn16, tables32g, mask_hybrid, seq, out32g, ws32g)
    torch.cuda.synchronize()
    seq.fill_(cfg.n_ctx)
    e0.record()
    for _ in range(16):
        lt.decode_step(shape32g, q32g, kn16, kn16, tables32g, mask_hybrid, seq, out32g, ws32g)
    e1.record()
    torch.cuda.synchronize()
    assert lt.check(ws32g) == 0
    ms = e0.elapsed_time(e1) / 16
    b32g = algorithmic_bytes_decode(cfg32g, n_mean, cfg.n_lazy)
    res["group_32"] = {"step_ms": ms, "decode_tokens_per_s": B / (ms * 1e-3), "gbs": b32g / (ms * 1e-3) / 1e9}
    del k16, v16, ks16, vs16, ws32g, tables32g
    # (e) fp32 caches (8 layers of the same head shape, every other one lazy): the CUDA-core kernels
    L32 = 8
    cfg32 = cfg.scaled(n_layers=L32, dtype="f32")
    shape32 = lt.Shape(L32, B, Hq, Hkv, D, cfg.n_sink, cfg.n_recent, cap, lt.LT_F32)
    mk32 = lambda n: [torch.randn((B, Hkv, n, D), device=dev) for _ in range(L32)]  # noqa: E731
    k32, v32, ks32, vs32 = mk32(cap), mk32(cap), mk32(C), mk32(C)
    tables32 = lt.LayerTables(shape32, k32, v32, ks32, vs32)
    ws32 = torch.empty(lt.workspace_bytes(shape32, cfg.n_ctx, T), dtype=torch.uint8, device=dev)
    lt.workspace_init(ws32)
    q32 = torch.randn((L32, B, Hq, D), device=dev)
    kn32 = torch.randn((L32, B, Hkv, D), device=dev)
    out32 = torch.zeros((L32, B, Hq, D), device=dev)
    mask32 = torch.zeros(L32, dtype=torch.uint8, device=dev)
    mask32[1::2] = 1
    seq = torch.full((B,), cfg.n_ctx, dtype=torch.int32, device=dev)
    for _ in range(2):
        lt.decode_step(shape32, q32, kn32, kn32, tables32, mask32, seq, out32, ws32)
    torch.cuda.synchronize()
    seq.fill_(cfg.n_ctx)
    e0.record()
    for _ in range(8):
        lt.decode_step(shape32, q32, kn32, kn32, tables32, mask32, seq, out32, ws32)
    e1.record()
    torch.cuda.synchronize()
    assert lt.check(ws32) == 0
    ms = e0.elapsed_time(e1) / 8
    b32 = algorithmic_bytes_decode(cfg32, cfg.n_ctx + 4.5, L32 // 2)
    res["fp32_caches_8_layers"] = {"step_ms": ms, "decode_tokens_per_s": B / (ms * 1e-3), "gbs": b32 / (ms * 1e-3) / 1e9,
                                   "frac_of_nominal_8TBs": b32 / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS}
    qt32 = torch.randn((L32, B, Hq, T, D), device=dev)
    sc32 = torch.zeros((L32, B, Hq), dtype=torch.float32, device=dev)
    lt.lazy_scores(shape32, qt32, tables32, cfg.n_ctx, T, sc32, ws32)
    torch.cuda.synchronize()
    e0.record()
    lt.lazy_scores(shape32, qt32, tables32, cfg.n_ctx, T, sc32, ws32)
    e1.record()
    torch.cuda.synchronize()
    assert lt.check(ws32) == 0
    ms = e0.elapsed_time(e1)
    res["fp32_caches_8_layers"]["lazy_scores_ms"] = ms
    res["fp32_caches_8_layers"]["lazy_scores_fp32_tflops"] = 2.0 * L32 * B * Hq * T * cfg.n_ctx * D / (ms * 1e-3) / 1e12
    del k32, v32, ks32, vs32, ws32, tables32, qt32
    return res


def _time_decode_steps(lt, shape, tables, mask, seq, n0, step_inputs, out, ws, steps, warm=3):
    """Mean ms of `steps` fused decode steps starting from length n0 (CUDA events on the current stream)."""
    seq.fill_(n0)
    for i in range(warm):
        q, k, v = step_inputs[i % len(step_inputs)]
        lt.decode_step(shape, q, k, v, tables, mask, seq, out, ws)
    torch.cuda.synchronize()
    seq.fill_(n0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        q, k, v = step_inputs[i % len(step_inputs)]
        lt.decode_step(shape, q, k, v, tables, mask, seq, out, ws)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def run_per_layer_calls(wl, mask_hybrid, peak, overlapped=False):
    """The deployment form of the step: a model calls the cache-updating attention once per layer (its other
    layers run in between), so a step is n_layers launches of one layer each; the last one advances seq_lens.
    overlapped: the same launches through lt_decode_step_layers, every launch but a step's first declared
    independent of the ones before it (this harness holds the inputs of all layers up front), so that a launch
    starts under the tail of the previous one."""
    cfg, lt = wl.cfg, wl.lt
    L, B = cfg.n_layers, cfg.batch
    steps = 12
    seq = torch.full((B,), cfg.n_ctx, dtype=torch.int32, device=wl.device)
    q, k, v = wl.step_inputs[0]
    ws = wl.ws
    if overlapped:
        ws = torch.empty(lt.workspace_bytes_layers(wl.shape, 0, 0), dtype=torch.uint8, device=wl.device)
        lt.workspace_init(ws)

    def one_step():
        for l in range(L):
            if overlapped:
                lt.decode_step_layers(wl.shape, q, k, v, wl.tables, mask_hybrid, seq, wl.out, ws, layer_begin=l,
                                      layer_count=1, advance_seq_lens=(l == L - 1), independent_of_previous=(l > 0))
            else:
                lt.decode_step(wl.shape, q, k, v, wl.tables, mask_hybrid, seq, wl.out, ws, layer_begin=l,
                               layer_count=1, advance_seq_lens=(l == L - 1))

    for _ in range(3):
        one_step()
    torch.cuda.synchronize()
    seq.fill_(cfg.n_ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one_step()
    e1.record()
    torch.cuda.synchronize()
    assert lt.check(ws) == 0
    ms = e0.elapsed_time(e1) / steps
    nbytes = float(np.mean([algorithmic_bytes_decode(cfg, cfg.n_ctx + i + 1, cfg.n_lazy) for i in range(steps)]))
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"launches_per_step": L, "step_ms": ms, "decode_tokens_per_s": B / (ms * 1e-3), "gbs": gbs,
            "frac_of_peak": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}


def run_other_configs(device, peak, gpu_index, only=None):
    """Throughput of the other paper-shaped workloads (detail only; the headline stays the 32K stack):
    the Llama-2-7B-shaped MHA 4K stack (hybrid against all-full), the Llama-3.1-8B-shaped 128K stack with
    the lazy fraction swept over 0 / 25 / 50 / 75 %, and the QwQ-32B-shaped long generation as a
    graph-replayed loop.  One stack lives on the device at a time."""
    import gc

    from synth import CONFIGS
    res = {}

    def step_metrics(cfg, ms, n_lazy, n_mean):
        nbytes = algorithmic_bytes_decode(cfg, n_mean, n_lazy)
        gbs = nbytes / (ms * 1e-3) / 1e9
        return {"step_ms": ms, "decode_tokens_per_s": cfg.batch / (ms * 1e-3), "algorithmic_bytes": nbytes, "gbs": gbs,
                "frac_of_peak": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}

    def score_ms(wl, iters=5):
        cfg, lt = wl.cfg, wl.lt
        for _ in range(2):
            lt.lazy_scores(wl.shape, wl.q_tail, wl.tables, cfg.n_ctx, cfg.w_last, wl.scores, wl.ws)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            lt.lazy_scores(wl.shape, wl.q_tail, wl.tables, cfg.n_ctx, cfg.w_last, wl.scores, wl.ws)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    # ---- Llama-2-7B-shaped MHA stack, 4K context ------------------------------------------------------
    def mha_4k():
        cfg = CONFIGS["llama2_7b_4k"]
        wl = Workload(cfg, device)
        lt = wl.lt
        steps = 16
        s_ms = score_ms(wl)
        wl.identify()
        torch.cuda.synchronize()
        assert sorted(np.nonzero(wl.mask.cpu().numpy())[0].tolist()) == wl.planted
        n_mean = cfg.n_ctx + (steps + 1) / 2
        hyb = _time_decode_steps(lt, wl.shape, wl.tables, wl.mask, wl.seq, cfg.n_ctx, wl.step_inputs, wl.out, wl.ws, steps)
        full_mask = torch.zeros_like(wl.mask)
        full = _time_decode_steps(lt, wl.shape, wl.tables, full_mask, wl.seq, cfg.n_ctx, wl.step_inputs, wl.out, wl.ws, steps)
        assert lt.check(wl.ws) == 0
        h, f = step_metrics(cfg, hyb, cfg.n_lazy, n_mean), step_metrics(cfg, full, 0, n_mean)
        return {"shape": "32 layers, 32 q / 32 kv heads (MHA), batch 32, context 4096, 16 lazy",
                "lazy_score_ms": s_ms, "hybrid": h, "all_full": f, "hybrid_over_all_full": full / hyb,
                "byte_ratio_ceiling": f["algorithmic_bytes"] / h["algorithmic_bytes"]}

    # ---- Llama-3.1-8B-shaped stack, 128K context, lazy fraction sweep ---------------------------------------
    def ctx_128k():
        cfg = CONFIGS["llama31_8b_128k"]
        wl = Workload(cfg, device)
        lt = wl.lt
        steps = 16
        L = cfg.n_layers
        s_ms = score_ms(wl)
        n_mean = cfg.n_ctx + (steps + 1) / 2
        sweep, base_ms = {}, None
        for n_lazy in (0, L // 4, L // 2, 3 * L // 4):
            lt.select_lazy(wl.scores, L, cfg.batch, cfg.n_q_heads, n_lazy, wl.mask)
            wl.seq.copy_(wl.seq0)
            lt.stream_init(wl.shape, wl.mask, wl.tables, wl.seq, ws=wl.ws)
            ms = _time_decode_steps(lt, wl.shape, wl.tables, wl.mask, wl.seq, cfg.n_ctx, wl.step_inputs, wl.out, wl.ws, steps)
            m = step_metrics(cfg, ms, n_lazy, n_mean)
            if base_ms is None:
                base_ms, base_bytes = ms, m["algorithmic_bytes"]
            m["speedup_over_all_full"] = base_ms / ms
            m["byte_ratio_ceiling"] = base_bytes / m["algorithmic_bytes"]
            sweep[f"{100 * n_lazy // L}%_lazy"] = m
        assert lt.check(wl.ws) == 0
        return {"shape": "32 layers, 32 q / 8 kv heads, batch 2, context 131072, window 4 + 4092",
                "lazy_score_ms": s_ms, "lazy_fraction_sweep": sweep}

    # ---- QwQ-32B-shaped long generation: eager loop against a graph-replayed loop -------------------------
    def long_generation():
        cfg = CONFIGS["qwq32b_longgen"]
        wl = Workload(cfg, device)
        lt = wl.lt
        L, B = cfg.n_layers, cfg.batch
        n_steps, per_graph = 2048, 16
        g = np.random.default_rng(41)
        m = np.zeros(L, dtype=np.uint8); m[g.permutation(L)[:cfg.n_lazy]] = 1     # the prompt is shorter than the window:
        wl.mask.copy_(torch.from_numpy(m).to(device))                             # every ratio is 1, so the mask is given
        q, k, v = wl.step_inputs[0]

        def reset():
            wl.seq.copy_(wl.seq0)
            lt.stream_init(wl.shape, wl.mask, wl.tables, wl.seq, ws=wl.ws)

        reset()
        for _ in range(3):
            lt.decode_step(wl.shape, q, k, v, wl.tables, wl.mask, wl.seq, wl.out, wl.ws)
        torch.cuda.synchronize()
        reset()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_steps):
            lt.decode_step(wl.shape, q, k, v, wl.tables, wl.mask, wl.seq, wl.out, wl.ws)
        e1.record()
        torch.cuda.synchronize()
        eager_ms = e0.elapsed_time(e1)
        # one captured graph of 16 steps (the step reads lengths and mask from the device), replayed 128 times
        reset()
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for _ in range(per_graph):
                    lt.decode_step(wl.shape, q, k, v, wl.tables, wl.mask, wl.seq, wl.out, wl.ws)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        reset()
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        reset()
        e0.record()
        for _ in range(n_steps // per_graph):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        graph_ms = e0.elapsed_time(e1)
        assert lt.check(wl.ws) == 0 and wl.seq.cpu().tolist() == [cfg.n_ctx + n_steps] * B
        nbytes = float(np.mean([algorithmic_bytes_decode(cfg, cfg.n_ctx + i + 1, cfg.n_lazy) for i in range(n_steps)]))
        return {
            "shape": "64 layers, 40 q / 8 kv heads (group of 5), batch 4, prompt 1024, 32 lazy, window 4 + 4092",
            "decode_steps": n_steps, "context_from_to": [cfg.n_ctx, cfg.n_ctx + n_steps],
            "mean_algorithmic_bytes_per_step": nbytes,
            "eager": {"step_ms": eager_ms / n_steps, "decode_tokens_per_s": B * n_steps / (eager_ms * 1e-3),
                      "gbs": nbytes / (eager_ms / n_steps * 1e-3) / 1e9},
            "graph_replay": {"steps_per_graph": per_graph, "step_ms": graph_ms / n_steps,
                             "decode_tokens_per_s": B * n_steps / (graph_ms * 1e-3),
                             "gbs": nbytes / (graph_ms / n_steps * 1e-3) / 1e9,
                             "frac_of_peak": nbytes / (graph_ms / n_steps * 1e-3) / 1e9 / peak}}

    for name, fn in (("llama2_7b_4k", mha_4k), ("llama31_8b_128k", ctx_128k), ("qwq32b_longgen", long_generation)):
        if only is not None and only != name:
            continue
        try:
            res[name] = fn()                   # the stack lives in fn's frame: gone when it returns
        except torch.cuda.OutOfMemoryError as e:  # a smaller device: say so instead of failing the headline
            res[name] = {"skipped": f"out of device memory: {e}"[:200]}
        gc.collect(); torch.cuda.empty_cache()
    return res



def run_e2e(wl, passes):
    """Same pass through the C ABI with HOST buffers: every step hands pinned host
    q / k_new / v_new to lt_decode_step_host, which copies them in, runs the step
    and copies the output back; the caller waits for it before the next step."""
    cfg, lt = wl.cfg, wl.lt
    pin = lambda t: t.cpu().pin_memory()  # noqa: E731
    h_qtail = pin(wl.q_tail)
    h_steps = [tuple(pin(x) for x in s) for s in wl.step_inputs]
    h_out = torch.empty(wl.out.shape, dtype=wl.out.dtype).pin_memory()
    h_mask = torch.empty(cfg.n_layers, dtype=torch.uint8).pin_memory()
    d_q, d_k, d_v = (torch.empty_like(x) for x in wl.step_inputs[0])
    h2d = sum(x.numel() * x.element_size() for x in h_steps[0])
    d2h = h_out.numel() * h_out.element_size()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def one_pass():
        wl.q_tail.copy_(h_qtail, non_blocking=True)
        wl.identify()
        h_mask.copy_(wl.mask, non_blocking=True)
        for i in range(cfg.steps):
            hq, hk, hv = h_steps[i % len(h_steps)]
            lt.decode_step_host(wl.shape, hq, hk, hv, h_out, d_q, d_k, d_v, wl.out, wl.tables, wl.mask, wl.seq, wl.ws)
            torch.cuda.current_stream().synchronize()       # the caller consumes the step's result

    one_pass()
    torch.cuda.synchronize()
    t0.record()
    for _ in range(passes):
        one_pass()
    t1.record()
    torch.cuda.synchronize()
    per_pass_bytes_in = h_qtail.numel() * h_qtail.element_size()
    return {"ms_per_pass": t0.elapsed_time(t1) / passes, "h2d": h2d + per_pass_bytes_in / cfg.steps,
            "d2h": d2h + cfg.n_layers / cfg.steps}


# ----------------------------------------------------------------------------
# CPU oracle timing (reported baseline, not the target)
# ----------------------------------------------------------------------------
def _oracle_sample(cfg, get_unit, get_tail, budget_s=20.0):
    """Time the oracle on a bounded sample: (layer, b) decode units of both kinds
    and one (layer, b) scoring unit; scale to the whole pass by unit count."""
    from threadpoolctl import threadpool_limits

    from oracle import lt_oracle as O
    n = cfg.n_ctx + 1
    with threadpool_limits(limits=1):
        t_full, t_lazy, nf, nl = 0.0, 0.0, 0, 0
        t_start = time.perf_counter()
        while time.perf_counter() - t_start < budget_s * 0.5 and nf < 4:
            q, K, V = get_unit(nf, n)
            a = time.perf_counter(); O.full_attention(q, K, V); t_full += time.perf_counter() - a; nf += 1
            a = time.perf_counter(); O.streaming_attention(q, K, V, cfg.n_sink, cfg.n_recent)
            t_lazy += time.perf_counter() - a; nl += 1
        Qt, Kp = get_tail()
        t_rows = max(1, min(cfg.w_last, 4))                  # a few of the w_last tail rows, all heads
        a = time.perf_counter()
        O.lazy_scores(Qt[:, -t_rows:], Kp, cfg.n_sink, cfg.n_recent)
        t_score_unit = (time.perf_counter() - a) * cfg.w_last / t_rows
    L, B, T = cfg.n_layers, cfg.batch, cfg.steps
    step_s = (t_full / nf) * (L - cfg.n_lazy) * B + (t_lazy / nl) * cfg.n_lazy * B
    score_s = t_score_unit * L * B
    pass_s = score_s + T * step_s
    return {"value": B * T / pass_s, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{nf} full + {nl} lazy (layer,batch-row) decode units (all 32 heads, n={n}) and "
                      f"{t_rows}/{cfg.w_last} tail rows of one scoring unit, fp64 numpy limited to 1 thread, "
                      f"scaled linearly to {L}x{B} units x {T} steps + one scoring pass",
            "decode_step_s": step_s, "lazy_score_s": score_s}


def cpu_baseline(cfg, wl):
    def get_unit(i, n):
        l, b = i % cfg.n_layers, i % cfg.batch
        q = wl.step_inputs[0][0][l, b].double().cpu().numpy()
        K = wl.k_full[l][b, :, :n].double().cpu().numpy()
        V = wl.v_full[l][b, :, :n].double().cpu().numpy()
        return q, K, V

    def get_tail():
        return wl.q_tail[0, 0].double().cpu().numpy(), wl.k_full[0][0, :, :cfg.n_ctx].double().cpu().numpy()

    return _oracle_sample(cfg, get_unit, get_tail)


def run_one_other_workload(args):
    """`--workload NAME`: one of the other paper-shaped workloads alone (what the default run reports under
    `detail.other_configs`), as one JSON line.  The headline line is the default run's."""
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(0)
    from paper_2410_13846_b200 import build
    build.build_library()
    peak, peak_kind = _peaks()
    res = run_other_configs(torch.device("cuda", 0), peak, 0, only=args.workload)
    print(json.dumps({"workload": args.workload, "peak_gbs": peak, "peak_kind": f"of {peak_kind}", **res}))


def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank, _, world = _dist_env()
    if rank != 0:
        return
    from synth import CONFIGS, decode_inputs, make_layer, planted_layers
    cfg = CONFIGS[WORKLOAD]
    small = cfg.scaled(n_layers=1, batch=1)
    qt, K, V = make_layer(small, 0, True, "cpu", capacity=cfg.n_ctx + 1)
    q = decode_inputs(small, 0, "cpu")[0]

    def get_unit(i, n):
        return q[0, 0].double().numpy(), K[0, :, :n].double().numpy(), V[0, :, :n].double().numpy()

    def get_tail():
        return qt[0].double().numpy(), K[0, :, :cfg.n_ctx].double().numpy()

    Kst, W = max(1, args.steps), max(0, args.warmup)
    res = None
    vals = []
    for i in range(min(W, 1) + min(Kst, 2)):
        res = _oracle_sample(cfg, get_unit, get_tail, budget_s=12.0)
        if i >= min(W, 1):
            vals.append(res["value"])
    value = float(np.mean(vals))
    B, T = cfg.batch, cfg.steps
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": Kst,
            "warmup": W, "ms_per_step": B * T / value * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "note": "CPU fp64 oracle on a bounded sample, scaled by unit count"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": res["cores"], "kind": "oracle", "sample": res["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_profile_case(args):
    """Small case of the same kernels for profiler captures: 4 layers (2 lazy) of
    the benchmark's stack (about 5 GB on the device, K/V per step far above the
    L2), one warm-up pass and one pass of a few decode steps, nothing else."""
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    from paper_2410_13846_b200 import build
    build.build_library()
    from synth import CONFIGS
    cfg = CONFIGS[WORKLOAD].scaled(n_layers=4, n_lazy=2, steps=args.profile_case)
    wl = Workload(cfg, torch.device("cuda", 0))
    wl.full_pass()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    wl.full_pass()
    torch.cuda.synchronize()
    print(json.dumps({"profile_case": cfg.name, "layers": cfg.n_layers, "decode_steps": cfg.steps,
                      "pass_s": time.perf_counter() - t0, "mask": wl.mask.cpu().tolist()}))


def run_profile_case_fp8(args):
    """Small case with FP8 caches for profiler captures: 4 layers (2 lazy) of the
    benchmark's stack shape, byte caches with random codes (2.3 GB on the device),
    two scoring passes from the 8-bit keys and a few decode steps, nothing else."""
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from paper_2410_13846_b200 import build
    build.build_library()
    import paper_2410_13846_b200 as lt
    from synth import CONFIGS
    cfg = CONFIGS[WORKLOAD].scaled(n_layers=4, n_lazy=2)
    L, B, Hq, Hkv, D = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    C, cap = cfg.n_sink + cfg.n_recent, cfg.n_ctx + 64
    scales = torch.full((L, 2), 0.02, dtype=torch.float32, device=dev)
    shape = lt.Shape(L, B, Hq, Hkv, D, cfg.n_sink, cfg.n_recent, cap, lt.LT_BF16, kv_fp8=1, kv_scales=scales)
    mk = lambda n: [torch.randint(0, 120, (B, Hkv, n, D), dtype=torch.uint8, device=dev) for _ in range(L)]
    tables = lt.LayerTables(shape, mk(cap), mk(cap), mk(C), mk(C))
    ws = torch.empty(lt.workspace_bytes(shape, cfg.n_ctx, cfg.w_last), dtype=torch.uint8, device=dev)
    lt.workspace_init(ws)
    mask = torch.tensor([0, 1, 1, 0], dtype=torch.uint8, device=dev)
    seq = torch.full((B,), cfg.n_ctx, dtype=torch.int32, device=dev)
    q = torch.randn((L, B, Hq, D), device=dev).bfloat16()
    k = torch.randn((L, B, Hkv, D), device=dev).bfloat16()
    out = torch.zeros_like(q)
    q_tail = torch.randn((L, B, Hq, cfg.w_last, D), device=dev).bfloat16()
    scores = torch.zeros((L, B, Hq), dtype=torch.float32, device=dev)
    t0 = time.perf_counter()
    for _ in range(2):      # the scoring pass from the 8-bit keys (the second launch is the warm one)
        lt.lazy_scores(shape, q_tail, tables, cfg.n_ctx, cfg.w_last, scores, ws)
    for _ in range(args.profile_case_fp8):
        lt.decode_step(shape, q, k, k, tables, mask, seq, out, ws)
    torch.cuda.synchronize()
    assert lt.check(ws) == 0
    print(json.dumps({"profile_case": "fp8 caches, " + cfg.name, "layers": L, "decode_steps": args.profile_case_fp8,
                      "run_s": time.perf_counter() - t0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default=None, choices=["llama2_7b_4k", "llama31_8b_128k", "qwq32b_longgen"],
                    help="run one of the other workloads alone and print its detail (not the headline line)")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the MHA 4K, long-generation and 128K workloads that are reported in `detail`")
    ap.add_argument("--profile-case", type=int, default=0, metavar="DECODE_STEPS",
                    help="run the 4-layer small case with this many decode steps per pass (for ncu) and exit")
    ap.add_argument("--profile-case-fp8", type=int, default=0, metavar="DECODE_STEPS",
                    help="run the 4-layer small case of the decode step with FP8 caches (for ncu) and exit")
    args = ap.parse_args()
    if args.profile_case_fp8 > 0:
        run_profile_case_fp8(args)
    elif args.profile_case > 0:
        run_profile_case(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.workload:
        run_one_other_workload(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
