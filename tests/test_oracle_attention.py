"""Pins for the oracle's attention functions (O1 full, O2 streaming).

Nothing here re-types the oracle's own formula: each test compares it with a
library routine, a closed form, an exact rational worked by hand, brute force
in pure Python, or an inequality the paper proves (Lemma F.4, Lemma F.1).
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import lt_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "log_integer_logits.txt")


def _rng(seed):
    return np.random.default_rng(seed)


def _golden_rows():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        n, s, r, fo, so, lm = line.split()
        rows.append((int(n), int(s), int(r), Fraction(fo), Fraction(so), Fraction(lm)))
    return rows


# ---- exact rationals worked by hand (Appendix E definition; Eq. 1) --------
@pytest.mark.parametrize("n,S,R,full_out,stream_out,mass", _golden_rows())
def test_log_integer_logits_golden(n, S, R, full_out, stream_out, mass):
    q = np.array([[1.0]])
    K = np.log(np.arange(1, n + 1, dtype=np.float64)).reshape(1, n, 1)
    V = np.arange(1, n + 1, dtype=np.float64).reshape(1, n, 1)
    assert abs(O.full_attention(q, K, V, scale=1.0)[0, 0] - float(full_out)) < 1e-12
    assert abs(O.streaming_attention(q, K, V, S, R, scale=1.0)[0, 0] - float(stream_out)) < 1e-12
    sc = O.lazy_scores(q.reshape(1, 1, 1), K, S, R, scale=1.0)
    assert abs(sc[0] - float(mass)) < 1e-12


# ---- library special case: torch float64 SDPA -----------------------------
@pytest.mark.parametrize("Hq,Hkv,n,D", [(4, 2, 37, 64), (8, 8, 5, 16), (5, 1, 130, 128), (10, 2, 64, 32)])
def test_full_attention_matches_torch_sdpa(Hq, Hkv, n, D):
    g = _rng(1)
    q = g.standard_normal((Hq, D))
    K = g.standard_normal((Hkv, n, D))
    V = g.standard_normal((Hkv, n, D))
    G = Hq // Hkv
    tq = torch.from_numpy(q)[None, :, None, :]                       # [1,Hq,1,D]
    tk = torch.from_numpy(K).repeat_interleave(G, dim=0)[None]       # [1,Hq,n,D]
    tv = torch.from_numpy(V).repeat_interleave(G, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0, :, 0, :].numpy()
    out = O.full_attention(q, K, V)
    assert np.max(np.abs(out - ref)) < 1e-12
    # a non-default scale goes through the same path
    ref2 = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.37)[0, :, 0, :].numpy()
    assert np.max(np.abs(O.full_attention(q, K, V, scale=0.37) - ref2)) < 1e-12


@pytest.mark.parametrize("n,S,R", [(50, 4, 10), (50, 0, 7), (9, 4, 60), (33, 3, 1), (200, 4, 60)])
def test_streaming_attention_matches_masked_sdpa(n, S, R):
    g = _rng(2)
    Hq, Hkv, D = 6, 3, 32
    q = g.standard_normal((Hq, D))
    K = g.standard_normal((Hkv, n, D))
    V = g.standard_normal((Hkv, n, D))
    # the mask is built here independently of the oracle's helper
    keep = torch.tensor([(j < S) or (j >= n - R) for j in range(n)])
    tq = torch.from_numpy(q)[None, :, None, :]
    tk = torch.from_numpy(K).repeat_interleave(2, dim=0)[None]
    tv = torch.from_numpy(V).repeat_interleave(2, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq, tk, tv, attn_mask=keep[None, None, None, :])[0, :, 0, :].numpy()
    out = O.streaming_attention(q, K, V, S, R)
    assert np.max(np.abs(out - ref)) < 1e-12


# ---- brute force in pure Python on tiny inputs ----------------------------
def _brute_attention(q, K, V, G, scale, keep=None):
    Hq, D = len(q), len(q[0])
    out = []
    for hq in range(Hq):
        g = hq // G
        n = len(K[g])
        logits = [scale * math.fsum(q[hq][d] * K[g][j][d] for d in range(D)) for j in range(n)]
        idx = [j for j in range(n) if keep is None or keep[j]]
        mx = max(logits[j] for j in idx)
        w = {j: math.exp(logits[j] - mx) for j in idx}
        Z = math.fsum(w.values())
        out.append([math.fsum(w[j] / Z * V[g][j][d] for j in idx) for d in range(D)])
    return out


@pytest.mark.parametrize("seed", range(6))
def test_full_and_streaming_brute_force(seed):
    g = _rng(100 + seed)
    Hkv = int(g.integers(1, 3))
    G = int(g.integers(1, 4))
    n = int(g.integers(1, 9))
    D = int(g.integers(1, 5))
    S = int(g.integers(0, 4))
    R = int(g.integers(1, 5))
    q = g.standard_normal((Hkv * G, D))
    K = g.standard_normal((Hkv, n, D))
    V = g.standard_normal((Hkv, n, D))
    sc = 1.0 / math.sqrt(D)
    bf = np.array(_brute_attention(q.tolist(), K.tolist(), V.tolist(), G, sc))
    assert np.max(np.abs(O.full_attention(q, K, V) - bf)) < 1e-13
    keep = [(j < S) or (j >= n - R) for j in range(n)]
    bs = np.array(_brute_attention(q.tolist(), K.tolist(), V.tolist(), G, sc, keep))
    assert np.max(np.abs(O.streaming_attention(q, K, V, S, R) - bs)) < 1e-13


# ---- closed forms ----------------------------------------------------------
def test_zero_query_gives_mean_of_values():
    g = _rng(3)
    K = g.standard_normal((2, 19, 8))
    V = g.standard_normal((2, 19, 8))
    out = O.full_attention(np.zeros((4, 8)), K, V)
    for hq in range(4):
        assert np.allclose(out[hq], V[hq // 2].mean(axis=0), atol=1e-14)
    # streaming: mean over the kept rows only
    S, R = 2, 5
    outs = O.streaming_attention(np.zeros((4, 8)), K, V, S, R)
    kept = list(range(S)) + list(range(19 - R, 19))
    for hq in range(4):
        assert np.allclose(outs[hq], V[hq // 2][kept].mean(axis=0), atol=1e-14)


def test_dominant_key_selects_its_value_row():
    g = _rng(4)
    D, n = 16, 40
    q = g.standard_normal((2, D))
    K = 0.01 * g.standard_normal((1, n, D))
    V = g.standard_normal((1, n, D))
    K[0, 17] = 400.0 * q[0] / np.dot(q[0], q[0])    # logit 400*scale for head 0
    out = O.full_attention(q, K, V, scale=1.0)
    assert np.max(np.abs(out[0] - V[0, 17])) < 1e-10
    # the GQA map is hq // G: head 1 reads the same kv head 0 (G = 2)
    K2 = 0.01 * g.standard_normal((2, n, D))
    V2 = g.standard_normal((2, n, D))
    q4 = g.standard_normal((4, D))
    K2[1, 5] = 400.0 * q4[3] / np.dot(q4[3], q4[3])
    out4 = O.full_attention(q4, K2, V2, scale=1.0)
    assert np.max(np.abs(out4[3] - V2[1, 5])) < 1e-10


def test_default_scale_is_inverse_sqrt_head_dim():
    # two keys, q.k = (a, 0): weights are sigmoid(+-a/sqrt(D))
    D = 64
    q = np.zeros((1, D)); q[0, 0] = 8.0
    K = np.zeros((1, 2, D)); K[0, 0, 0] = 2.0           # q.k0 = 16, q.k1 = 0
    V = np.zeros((1, 2, D)); V[0, 0, 0] = 1.0
    out = O.full_attention(q, K, V)
    assert abs(out[0, 0] - 1.0 / (1.0 + math.exp(-16.0 / 8.0))) < 1e-14


# ---- invariants ------------------------------------------------------------
def test_softmax_rows_sum_to_one_and_lipschitz():
    g = _rng(5)
    for _ in range(20):
        x = 10 * g.standard_normal(57)
        y = x + 0.3 * g.standard_normal(57)
        px, py = O.softmax(x), O.softmax(y)
        assert abs(px.sum() - 1.0) < 1e-12 and np.all(px >= 0)
        # Lemma F.1: ||sm(x) - sm(y)||_1 <= 2 ||x - y||_inf
        assert np.abs(px - py).sum() <= 2 * np.max(np.abs(x - y)) + 1e-12
    # shift invariance and no overflow at large logits
    x = g.standard_normal(9)
    assert np.allclose(O.softmax(x + 1000.0), O.softmax(x), atol=1e-13)


@pytest.mark.parametrize("n,S,R", [(10, 4, 6), (10, 4, 60), (3, 4, 1), (1, 0, 1), (64, 0, 64)])
def test_streaming_equals_full_when_window_covers_history(n, S, R):
    assert S + R >= n
    g = _rng(6)
    q = g.standard_normal((4, 16))
    K = g.standard_normal((2, n, 16))
    V = g.standard_normal((2, n, 16))
    a = O.full_attention(q, K, V)
    b = O.streaming_attention(q, K, V, S, R)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("seed", range(5))
def test_lemma_f4_equality_and_bound(seed):
    """Lemma F.4: with K1 the kept keys and K2 the discarded ones,
    ||s1 - s1~||_1 = ||s2||_1 and the outputs differ by at most
    2 ||s2||_1 max(||V1||_{2,inf}, ||V2||_{2,inf}).  ||s2||_1 is 1 - lazy mass
    (Eq. 1 with one tail query), so the three oracle functions are tied together.
    """
    g = _rng(200 + seed)
    n, D, S, R = 90, 24, 3, 11
    q = g.standard_normal((1, D))
    K = g.standard_normal((1, n, D))
    V = g.standard_normal((1, n, D))
    full = O.full_attention(q, K, V)[0]
    stream = O.streaming_attention(q, K, V, S, R)[0]
    mass = O.lazy_scores(q.reshape(1, 1, D), K, S, R)[0]
    s2 = 1.0 - mass
    vmax = np.max(np.linalg.norm(V[0], axis=1))
    assert np.linalg.norm(stream - full) <= 2 * s2 * vmax + 1e-12
    # the equality: with the identity as value matrix the output *is* the
    # attention-weight vector
    eye = np.eye(n)[None]
    w_full = O.full_attention(q, K, eye)[0]
    w_str = O.streaming_attention(q, K, eye, S, R)[0]
    kept = np.array([(j < S) or (j >= n - R) for j in range(n)])
    assert abs(np.abs(w_full[kept] - w_str[kept]).sum() - w_full[~kept].sum()) < 1e-12
    assert abs(w_full[~kept].sum() - s2) < 1e-12
    assert np.all(w_str[~kept] == 0.0)


def test_planted_mistakes_are_caught():
    """A transposed operand, a dropped scale or a wrong GQA map must fail the
    SDPA pin: mutate a copy of the inputs the way such a bug would and check the
    results really differ by far more than the pin's tolerance."""
    g = _rng(7)
    Hq, Hkv, n, D = 4, 2, 21, 8
    q = g.standard_normal((Hq, D)); K = g.standard_normal((Hkv, n, D)); V = g.standard_normal((Hkv, n, D))
    good = O.full_attention(q, K, V)
    assert np.max(np.abs(O.full_attention(q, K, V, scale=1.0) - good)) > 1e-3          # dropped scale
    assert np.max(np.abs(O.full_attention(q[[0, 2, 1, 3]], K, V)[[0, 2, 1, 3]] - good)) > 1e-3  # hq % Hkv map
    assert np.max(np.abs(O.full_attention(q, K[:, ::-1], V) - good)) > 1e-3            # index reversal
