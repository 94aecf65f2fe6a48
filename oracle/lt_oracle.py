"""fp64 CPU oracle for the LightTransfer hybrid decode-attention path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain reference that the
CUDA library is checked against.  Nothing on the product path may import it:
only the tests, the smoke check and the benchmark's CPU-baseline leg do.  It
shares no code with the CUDA path and imports nothing from it.

Every function works in float64 on numpy arrays and follows the definitions in
the paper one step at a time, with no blocking, fusion or reordering:

  O1  full_attention        causal softmax attention, decode form (Appendix E,
                            definition of the self-attention module and mask M;
                            Section 3, "Inference stages")
  O2  streaming_attention   the same with the sink+recent mask M_lazy
                            (Appendix E, masked MHA; Section 5.1, retained KV)
  O3  lazy_scores           the lazy ratio of Eq. 1, per query head; a second
                            route through the log-sum-exp identity of Table 1;
                            causal_lse / lazy_scores_from_lse: the form Section
                            5.1 actually deploys - the prefill's log-sum-exp is
                            given, only the window block is recomputed
  O4  select_lazy           keep the P lowest ratios full (Section 5.1, the
                            priority queue; Figure 3)
  O5  ring_slot / ring_owner / stream_cache_after / HybridReplay
                            integer model of the constant-size cache of a lazy
                            layer (Section 5.1, retained {X_initial, X_recent})
  O6  quantize_e4m3         8-bit storage of cached keys / values (not in the
                            paper, which keeps BF16 everywhere, Appendix A; an
                            adjacent deployment option): the OCP FP8 E4M3
                            format written out from its definition

Readings taken where the paper is silent or inconsistent (scale 1/sqrt(D) in
numerator and denominator, causal mask inside the tail block, X_recent as the
fixed last w_recent prompt positions, set union of sink and recent, contiguous
GQA groups, mean of ratios and never of their logarithms, append-then-attend)
are listed in the design notes of the repository.

Pins (see tests/test_oracle_*.py): torch float64 scaled_dot_product_attention
as a library special case, closed forms for q = 0 and for logits that are
logarithms of integers, brute force on tiny inputs, Lemma F.4's equality and
bound, ratio == 1 when the window covers every key, exhaustive ring replay.
No function here is "parity unpinned".
"""
from __future__ import annotations

import heapq
import math

import numpy as np

__all__ = [
    "softmax",
    "full_attention",
    "streaming_attention",
    "kept_positions",
    "lazy_scores",
    "lazy_scores_lse_route",
    "causal_lse",
    "lazy_scores_from_lse",
    "layer_ratios",
    "select_lazy",
    "select_lazy_priority_queue",
    "select_lazy_priority_queue_trace",
    "select_lazy_per_sequence",
    "select_lazy_by_frequency",
    "lazy_scores_per_row_window",
    "ring_slot",
    "ring_valid_slots",
    "ring_owner",
    "stream_cache_after",
    "HybridReplay",
    "e4m3_values",
    "quantize_e4m3",
]


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def _default_scale(head_dim: int, scale) -> float:
    # The paper's theory drops the scale and Table 1 mixes a scaled lse with an
    # unscaled matmul; 1/sqrt(D) on both sides is the self-consistent reading.
    if scale is None or scale <= 0:
        return 1.0 / math.sqrt(head_dim)
    return float(scale)


def softmax(x):
    """Row softmax of a 1-D vector, max-subtracted (Appendix E, sm(.))."""
    x = _f64(x)
    e = np.exp(x - np.max(x))
    return e / np.sum(e)


# --------------------------------------------------------------------------
# O1 / O2: one decode step of one layer and one batch row
# --------------------------------------------------------------------------
def full_attention(q, K, V, scale=None):
    """O1.  out[hq] = softmax(scale * q[hq] . K[g]^T) V[g],  g = hq // G.

    q: [Hq, D]   the query of the token being decoded (already in the cache:
                 the causal mask has i >= j, so the newest key is visible)
    K: [Hkv, n, D], V: [Hkv, n, Dv]   every cached key / value of this layer
                 and batch row (Dv = D in every model; kept separate as in
                 the paper's W_V)
    returns out [Hq, Dv].
    (Appendix E, att(X, W_Q, W_K, W_V) with the causal mask M, last row.)
    """
    q, K, V = _f64(q), _f64(K), _f64(V)
    Hq, D = q.shape
    Hkv, n, _ = K.shape
    assert Hq % Hkv == 0 and n >= 1
    G = Hq // Hkv
    sc = _default_scale(D, scale)
    out = np.zeros((Hq, V.shape[2]), dtype=np.float64)
    for hq in range(Hq):
        g = hq // G
        s = sc * (K[g] @ q[hq])          # logits over keys 0..n-1
        p = softmax(s)
        out[hq] = p @ V[g]
    return out


def kept_positions(n: int, n_sink: int, n_recent: int):
    """Boolean vector over positions 0..n-1: True where the key is kept by a
    lazy layer, i.e. j < n_sink or j >= n - n_recent (a set union, so an
    overlap is not counted twice).  (Section 5.1; Appendix E: the first 4 and the last
    1020 tokens in the paper's setting.)
    """
    j = np.arange(n)
    return (j < n_sink) | (j >= n - n_recent)


def streaming_attention(q, K, V, n_sink: int, n_recent: int, scale=None):
    """O2.  O1 with every logit outside the kept set at -inf.

    Evaluated on the logical, complete history K, V [Hkv, n, D] with an index
    predicate; no ring buffer is involved here.
    (Appendix E, masked MHA with M_lazy.)
    """
    q, K, V = _f64(q), _f64(K), _f64(V)
    Hq, D = q.shape
    Hkv, n, _ = K.shape
    assert Hq % Hkv == 0 and n >= 1
    G = Hq // Hkv
    sc = _default_scale(D, scale)
    keep = kept_positions(n, n_sink, n_recent)
    out = np.zeros((Hq, V.shape[2]), dtype=np.float64)
    for hq in range(Hq):
        g = hq // G
        s = sc * (K[g] @ q[hq])
        s = np.where(keep, s, -np.inf)
        p = softmax(s)
        out[hq] = p @ V[g]
    return out


# --------------------------------------------------------------------------
# O3: the lazy ratio of Eq. 1
# --------------------------------------------------------------------------
def lazy_scores(Q_tail, K, n_sink: int, n_recent: int, scale=None):
    """O3.  Per-query-head lazy ratio of one layer and one batch row (Eq. 1).

    Q_tail: [Hq, T, D]  queries of the last T = w_last prompt positions
                        n-T .. n-1
    K:      [Hkv, n, D] prompt keys
    For tail query t at position i = n - T + t the attention row is the causal
    softmax over keys 0..i; its mass on {j < n_sink} U {j >= n - n_recent} is
    summed and the T masses are averaged.  returns score [Hq] in [0, 1].
    The average over heads that completes Eq. 1 is taken in layer_ratios().
    """
    Q_tail, K = _f64(Q_tail), _f64(K)
    Hq, T, D = Q_tail.shape
    Hkv, n, _ = K.shape
    assert Hq % Hkv == 0 and 1 <= T <= n
    G = Hq // Hkv
    sc = _default_scale(D, scale)
    keep = kept_positions(n, n_sink, n_recent)
    score = np.zeros(Hq, dtype=np.float64)
    for hq in range(Hq):
        g = hq // G
        acc = 0.0
        for t in range(T):
            i = n - T + t
            s = sc * (K[g, : i + 1] @ Q_tail[hq, t])
            p = softmax(s)
            acc += float(np.sum(p[keep[: i + 1]]))
        score[hq] = acc / T
    return score


def _logsumexp(x):
    x = _f64(x)
    if x.size == 0:
        return -np.inf
    m = np.max(x)
    if not np.isfinite(m):
        return m
    return m + math.log(float(np.sum(np.exp(x - m))))


def lazy_scores_lse_route(Q_tail, K, n_sink: int, n_recent: int, scale=None):
    """O3, second route (Table 1): ratio = exp(lse(window logits) - lse(all
    visible logits)), exponentiated before averaging over the tail queries.
    Must agree with lazy_scores() to rounding.
    """
    Q_tail, K = _f64(Q_tail), _f64(K)
    Hq, T, D = Q_tail.shape
    Hkv, n, _ = K.shape
    G = Hq // Hkv
    sc = _default_scale(D, scale)
    keep = kept_positions(n, n_sink, n_recent)
    score = np.zeros(Hq, dtype=np.float64)
    for hq in range(Hq):
        g = hq // G
        acc = 0.0
        for t in range(T):
            i = n - T + t
            s = sc * (K[g, : i + 1] @ Q_tail[hq, t])
            lse_all = _logsumexp(s)
            lse_win = _logsumexp(s[keep[: i + 1]])
            acc += math.exp(lse_win - lse_all) if np.isfinite(lse_win) else 0.0
        score[hq] = acc / T
    return score


def causal_lse(Q_tail, K, scale=None):
    """What the prefill's attention hands over for the tail rows (Table 1, the
    `lse` returned next to `attn_out`): lse[hq, t] = log sum_{j <= i} exp(scale *
    q_t . k_j), natural logarithm, i = n - T + t.  returns [Hq, T].
    """
    Q_tail, K = _f64(Q_tail), _f64(K)
    Hq, T, D = Q_tail.shape
    Hkv, n, _ = K.shape
    G = Hq // Hkv
    sc = _default_scale(D, scale)
    out = np.zeros((Hq, T), dtype=np.float64)
    for hq in range(Hq):
        for t in range(T):
            i = n - T + t
            out[hq, t] = _logsumexp(sc * (K[hq // G, : i + 1] @ Q_tail[hq, t]))
    return out


def lazy_scores_from_lse(Q_tail, K, lse, n_sink: int, n_recent: int, scale=None):
    """O3 as deployed (Section 5.1: with the prefill's denominators at hand only
    the window block is recomputed; Table 1): the denominator of every tail row comes in as
    its log-sum-exp, and only the logits of the kept keys {j < n_sink} U
    {j >= n - n_recent} (causally visible ones) are computed:
        mass_t = sum_{j kept, j <= i} exp(scale * q_t . k_j - lse[hq, t]),
    averaged over the T tail rows.  K is the whole prompt [Hkv, n, D] only so
    that positions can be indexed; rows outside the kept set are not touched.
    """
    Q_tail, K, lse = _f64(Q_tail), _f64(K), _f64(lse)
    Hq, T, D = Q_tail.shape
    Hkv, n, _ = K.shape
    G = Hq // Hkv
    sc = _default_scale(D, scale)
    kept = np.nonzero(kept_positions(n, n_sink, n_recent))[0]
    score = np.zeros(Hq, dtype=np.float64)
    for hq in range(Hq):
        acc = 0.0
        for t in range(T):
            i = n - T + t
            js = kept[kept <= i]
            logits = sc * (K[hq // G, js] @ Q_tail[hq, t])
            acc += float(np.sum(np.exp(logits - lse[hq, t])))
        score[hq] = acc / T
    return score


def lazy_scores_per_row_window(Q_tail, K, n_sink: int, n_recent: int, scale=None):
    """O3 under the other reading of X_recent (Appendix E: the mask M_lazy keeps,
    for row i, the first few and the most recent tokens of [i]): the recent set of
    the tail query at position i is {i - n_recent + 1 .. i} instead of the fixed
    block {n - n_recent .. n - 1}.  Both readings agree for the last query.
    """
    Q_tail, K = _f64(Q_tail), _f64(K)
    Hq, T, D = Q_tail.shape
    Hkv, n, _ = K.shape
    assert Hq % Hkv == 0 and 1 <= T <= n
    G = Hq // Hkv
    sc = _default_scale(D, scale)
    score = np.zeros(Hq, dtype=np.float64)
    for hq in range(Hq):
        acc = 0.0
        for t in range(T):
            i = n - T + t
            s = sc * (K[hq // G, : i + 1] @ Q_tail[hq, t])
            p = softmax(s)
            j = np.arange(i + 1)
            acc += float(np.sum(p[(j < n_sink) | (j > i - n_recent)]))
        score[hq] = acc / T
    return score


# --------------------------------------------------------------------------
# O4: selection
# --------------------------------------------------------------------------
def layer_ratios(scores):
    """r_l = mean over batch rows and query heads of scores[l] (Eq. 1's average
    over heads; Figure 2 averages over the samples of a batch)."""
    scores = _f64(scores)
    L = scores.shape[0]
    return scores.reshape(L, -1).mean(axis=1)


def select_lazy(scores, n_lazy: int):
    """O4.  mask[l] = 1 for the n_lazy layers with the largest ratio; ties go
    to the lower layer index.  Equivalently the P = L - n_lazy lowest ratios
    keep full attention (Section 5.1).  returns (mask uint8 [L], r float64 [L]).
    """
    r = layer_ratios(scores)
    L = r.shape[0]
    assert 0 <= n_lazy <= L
    order = sorted(range(L), key=lambda l: (-r[l], l))
    mask = np.zeros(L, dtype=np.uint8)
    for l in order[:n_lazy]:
        mask[l] = 1
    return mask, r


def select_lazy_priority_queue(ratios, n_full: int):
    """O4, literal form (Section 5.1, Figure 3): walk the layers in order, push
    (ratio, layer) into a max-priority queue of capacity P = n_full; whenever
    the queue holds more than P entries pop the largest ratio and label that
    layer lazy.  Equal ratios pop the lower layer first.  returns mask [L].
    """
    ratios = _f64(ratios)
    L = ratios.shape[0]
    assert 0 <= n_full <= L
    mask = np.zeros(L, dtype=np.uint8)
    heap = []  # heapq is a min-heap: store (-ratio, layer)
    for l in range(L):
        heapq.heappush(heap, (-ratios[l], l))
        if len(heap) > n_full:
            _, popped = heapq.heappop(heap)
            mask[popped] = 1
    return mask


def select_lazy_priority_queue_trace(ratios, n_full: int):
    """The same queue, one layer at a time (Figure 3): popped[l] is the layer
    that leaves the queue - and becomes lazy, its KV reduced at once - when
    layer l arrives, or -1 while the queue still has room.  returns (mask, popped).
    """
    ratios = _f64(ratios)
    L = ratios.shape[0]
    mask = np.zeros(L, dtype=np.uint8)
    popped = np.full(L, -1, dtype=np.int64)
    queue = []  # layers currently held, kept as a plain list: the definition, not a heap
    for l in range(L):
        queue.append(l)
        if len(queue) > n_full:
            top = max(queue, key=lambda m: (ratios[m], -m))  # highest ratio, lower index on ties
            queue.remove(top)
            mask[top] = 1
            popped[l] = top
    return mask, popped


def select_lazy_per_sequence(scores, n_lazy: int):
    """O4 per prompt (Section 4: which layers are lazy differs from prompt to
    prompt): row b of the result is select_lazy on that batch row's scores
    alone.  scores [L, B, Hq] -> mask uint8 [B, L], r float64 [B, L].
    """
    scores = _f64(scores)
    L, B, _ = scores.shape
    mask = np.zeros((B, L), dtype=np.uint8)
    r = np.zeros((B, L), dtype=np.float64)
    for b in range(B):
        mask[b], r[b] = select_lazy(scores[:, b : b + 1, :], n_lazy)
    return mask, r


def select_lazy_by_frequency(masks, n_lazy: int):
    """Layer choice of LightTransfer-Train (Section 5.2): every training sample
    labels its own lazy layers; count, per layer, how many samples labelled it
    lazy and keep the n_lazy layers with the highest counts (lower index on
    ties).  masks [N, L] of 0/1 -> (mask uint8 [L], counts int64 [L]).
    """
    masks = np.asarray(masks)
    N, L = masks.shape
    assert 0 <= n_lazy <= L
    counts = np.zeros(L, dtype=np.int64)
    for i in range(N):
        for l in range(L):
            counts[l] += 1 if masks[i, l] else 0
    order = sorted(range(L), key=lambda l: (-counts[l], l))
    out = np.zeros(L, dtype=np.uint8)
    for l in order[:n_lazy]:
        out[l] = 1
    return out, counts


# --------------------------------------------------------------------------
# O5: integer model of the constant-size cache
# --------------------------------------------------------------------------
def ring_slot(p: int, n_sink: int, n_recent: int) -> int:
    """Slot of token position p in a lazy layer's cache of n_sink + n_recent
    rows: sinks keep their own row, later tokens cycle through the ring."""
    if p < n_sink:
        return p
    return n_sink + (p - n_sink) % n_recent


def ring_valid_slots(n: int, n_sink: int, n_recent: int) -> int:
    """Rows in use after n tokens."""
    return min(n, n_sink) + min(max(n - n_sink, 0), n_recent)


def ring_owner(s: int, n: int, n_sink: int, n_recent: int):
    """Largest position p < n that was written to slot s, or None."""
    owner = None
    for p in range(n):
        if ring_slot(p, n_sink, n_recent) == s:
            owner = p
    return owner


def stream_cache_after(hist, n_sink: int, n_recent: int):
    """Replay: write rows hist[0], hist[1], ... one by one at their slots and
    return (cache [n_sink + n_recent, ...], valid_rows).  hist: [n, ...] with
    any trailing shape and any dtype (bit patterns are carried unchanged)."""
    hist = np.asarray(hist)
    n = hist.shape[0]
    cache = np.zeros((n_sink + n_recent,) + hist.shape[1:], dtype=hist.dtype)
    for p in range(n):
        cache[ring_slot(p, n_sink, n_recent)] = hist[p]
    return cache, ring_valid_slots(n, n_sink, n_recent)


class HybridReplay:
    """Sequence replay of one batch row: keeps the complete logical history of
    every layer and, after each append, evaluates O1 (mask 0) or O2 (mask 1).
    The new token attends to itself: append first, then attend.
    """

    def __init__(self, layer_mask, n_sink: int, n_recent: int, scale=None):
        self.mask = [int(m) for m in layer_mask]
        self.S, self.R, self.scale = n_sink, n_recent, scale
        self.K = [None] * len(self.mask)   # per layer [Hkv, n, D]
        self.V = [None] * len(self.mask)

    def load_prompt(self, l: int, K, V):
        self.K[l] = _f64(K).copy()
        self.V[l] = _f64(V).copy()

    def append(self, l: int, k_new, v_new):
        k_new, v_new = _f64(k_new), _f64(v_new)        # [Hkv, D]
        self.K[l] = np.concatenate([self.K[l], k_new[:, None, :]], axis=1)
        self.V[l] = np.concatenate([self.V[l], v_new[:, None, :]], axis=1)

    def attend(self, l: int, q):
        if self.mask[l]:
            return streaming_attention(q, self.K[l], self.V[l], self.S, self.R, self.scale)
        return full_attention(q, self.K[l], self.V[l], self.scale)


# --------------------------------------------------------------------------
# O6: FP8 E4M3 storage (OCP 8-bit floating point specification, E4M3 variant)
# --------------------------------------------------------------------------
def e4m3_values():
    """Value of every E4M3 code 0..255 as float64 (NaN for the two NaN codes).
    Layout s.eeee.mmm, exponent bias 7; e = 0 is subnormal (m/8 * 2^-6); there
    are no infinities, and s.1111.111 is NaN, so the largest finite value is
    1.75 * 2^8 = 448."""
    out = np.zeros(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e = (code >> 3) & 0xF
        m = code & 0x7
        if e == 0xF and m == 0x7:
            out[code] = np.nan
        elif e == 0:
            out[code] = sign * (m / 8.0) * 2.0 ** -6
        else:
            out[code] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return out


def quantize_e4m3(x, scale):
    """Codes and dequantised values of x stored as E4M3 with one scale:
        y = float32(x) / float32(scale)          (one IEEE float32 division)
        code = nearest E4M3 value to y, ties to the even code, saturating at +-448
        value = E4M3(code) * float32(scale)      (exact in float64)
    NaN maps to the NaN code.  returns (codes uint8, values float64), shaped like x.
    """
    table = e4m3_values()
    xs = np.asarray(x, dtype=np.float32)
    y = (xs / np.float32(scale)).astype(np.float32).astype(np.float64)
    flat = y.reshape(-1)
    codes = np.zeros(flat.shape, dtype=np.uint8)
    pos_codes = np.arange(0, 0x7F)               # 0 .. 126: non-negative finite values, increasing
    pos_vals = table[pos_codes]
    for i, v in enumerate(flat):
        if np.isnan(v):
            codes[i] = 0x7F
            continue
        a = min(abs(v), 448.0)
        hi = int(np.searchsorted(pos_vals, a, side="left"))      # first value >= a
        if hi == 0:
            c = 0
        else:
            lo = hi - 1
            if hi >= len(pos_vals):
                c = lo
            else:
                dlo, dhi = a - pos_vals[lo], pos_vals[hi] - a
                if dlo < dhi:
                    c = lo
                elif dhi < dlo:
                    c = hi
                else:
                    c = lo if (lo & 1) == 0 else hi              # tie: even mantissa
        codes[i] = c | (0x80 if np.signbit(v) else 0)
    codes = codes.reshape(y.shape)
    values = table[codes] * float(np.float32(scale))
    return codes, values
