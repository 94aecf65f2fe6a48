"""Pins for the oracle's lazy ratio (O3), selection (O4) and ring model (O5)."""
import itertools
import math

import numpy as np
import pytest

from oracle import lt_oracle as O


def _rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- O3 --------
@pytest.mark.parametrize("n,S,R,T", [(40, 4, 36, 8), (40, 4, 60, 16), (7, 4, 4, 7), (12, 0, 12, 3)])
def test_ratio_is_one_when_window_covers_every_key(n, S, R, T):
    """Section 5.2: with a window large relative to the input the ratio stays at 1."""
    g = _rng(10)
    Q = g.standard_normal((4, T, 16))
    K = g.standard_normal((2, n, 16))
    sc = O.lazy_scores(Q, K, S, R)
    assert np.max(np.abs(sc - 1.0)) < 1e-12


@pytest.mark.parametrize("seed", range(4))
def test_two_routes_agree(seed):
    """Table 1's identity: ratio = exp(lse(window logits) - lse(all logits))."""
    g = _rng(20 + seed)
    n, T, D = 150, 9, 24
    Q = 2.0 * g.standard_normal((6, T, D))
    K = g.standard_normal((3, n, D))
    for S, R in [(4, 20), (0, 5), (3, 200), (4, 4)]:
        a = O.lazy_scores(Q, K, S, R)
        b = O.lazy_scores_lse_route(Q, K, S, R)
        assert np.max(np.abs(a - b)) < 1e-12
        assert np.all(a >= 0) and np.all(a <= 1 + 1e-15)


def test_causal_lse_matches_library_logsumexp_and_closed_forms():
    """The denominator handed over by the prefill: scipy's logsumexp as the
    library special case; q = 0 gives log(i + 1); logits that are logarithms of
    integers give the logarithm of their sum (tests/golden/log_integer_logits.txt)."""
    from scipy.special import logsumexp
    g = _rng(31)
    n, T, D = 90, 7, 12
    Q = 1.7 * g.standard_normal((4, T, D))
    K = g.standard_normal((2, n, D))
    lse = O.causal_lse(Q, K, 0.3)
    for hq in range(4):
        for t in range(T):
            i = n - T + t
            ref = logsumexp(0.3 * np.einsum("jd,d->j", K[hq // 2, : i + 1], Q[hq, t]))
            assert abs(lse[hq, t] - ref) < 1e-12
    z = O.causal_lse(np.zeros((2, T, D)), K)
    assert np.max(np.abs(z - np.log(np.arange(n - T + 1, n + 1))[None, :])) < 1e-13
    for n_ in (4, 6, 8):
        k = np.log(np.arange(1, n_ + 1, dtype=np.float64)).reshape(1, n_, 1)
        assert abs(O.causal_lse(np.ones((1, 1, 1)), k, 1.0)[0, 0] - math.log(n_ * (n_ + 1) / 2)) < 1e-13


@pytest.mark.parametrize("seed", range(3))
def test_scores_from_lse_equal_eq1_and_the_hand_worked_rationals(seed):
    """Recomputing only the window block against the given log-sum-exp is Eq. 1
    itself (Table 1's identity), including overlap of sink and window, no sink,
    and a tail longer than the window."""
    g = _rng(40 + seed)
    n, T, D = 130, 11, 20
    Q = 2.0 * g.standard_normal((6, T, D))
    K = g.standard_normal((3, n, D))
    for S, R, sc in [(4, 20, None), (0, 5, 0.2), (3, 200, None), (4, 4, None), (2, 7, 0.05)]:
        lse = O.causal_lse(Q, K, sc)
        a = O.lazy_scores(Q, K, S, R, sc)
        b = O.lazy_scores_from_lse(Q, K, lse, S, R, sc)
        assert np.max(np.abs(a - b)) < 1e-12
    # a wrong denominator shows: doubling exp(lse) halves every mass
    lse = O.causal_lse(Q, K)
    a = O.lazy_scores_from_lse(Q, K, lse, 4, 20)
    assert np.max(np.abs(O.lazy_scores_from_lse(Q, K, lse + math.log(2.0), 4, 20) - a / 2)) < 1e-13
    # hand-worked fixture: logits ln 1 .. ln n, lse = ln(n(n+1)/2), mass of the last query as a fraction
    import os
    from fractions import Fraction
    path = os.path.join(os.path.dirname(__file__), "golden", "log_integer_logits.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        n_, S, R, _, _, mass = line.split()
        n_, S, R = int(n_), int(S), int(R)
        k = np.log(np.arange(1, n_ + 1, dtype=np.float64)).reshape(1, n_, 1)
        lse1 = np.array([[math.log(n_ * (n_ + 1) / 2)]])
        got = O.lazy_scores_from_lse(np.ones((1, 1, 1)), k, lse1, S, R, 1.0)[0]
        assert abs(got - float(Fraction(mass))) < 1e-14


def _uniform_mass(n, S, R, T):
    """Closed form for q = 0 (uniform attention): the tail query at position i
    sees i+1 keys of which |{j<=i: j<S or j>=n-R}| are kept."""
    tot = 0.0
    for t in range(T):
        i = n - T + t
        kept = sum(1 for j in range(i + 1) if j < S or j >= n - R)
        tot += kept / (i + 1)
    return tot / T


@pytest.mark.parametrize("n,S,R,T", [(100, 4, 10, 16), (100, 4, 10, 5), (30, 0, 7, 30), (64, 6, 3, 8), (20, 4, 40, 4)])
def test_uniform_attention_closed_form(n, S, R, T):
    K = _rng(11).standard_normal((1, n, 8))
    sc = O.lazy_scores(np.zeros((2, T, 8)), K, S, R)
    assert np.max(np.abs(sc - _uniform_mass(n, S, R, T))) < 1e-13
    # closed form for one row when the window does not overlap the sinks:
    if S <= n - R:
        i = n - 1
        assert abs(_uniform_mass(n, S, R, 1) - (min(S, i + 1) + max(0, i - max(S, n - R) + 1)) / (i + 1)) < 1e-15


def _brute_lazy(Q, K, G, S, R, scale):
    Hq, T, D = len(Q), len(Q[0]), len(Q[0][0])
    n = len(K[0])
    res = []
    for hq in range(Hq):
        g = hq // G
        acc = 0.0
        for t in range(T):
            i = n - T + t
            lg = [scale * math.fsum(Q[hq][t][d] * K[g][j][d] for d in range(D)) for j in range(i + 1)]
            mx = max(lg)
            w = [math.exp(x - mx) for x in lg]
            Z = math.fsum(w)
            acc += math.fsum(w[j] for j in range(i + 1) if (j < S or j >= n - R)) / Z
        res.append(acc / T)
    return res


@pytest.mark.parametrize("seed", range(6))
def test_lazy_scores_brute_force(seed):
    g = _rng(30 + seed)
    Hkv, G = int(g.integers(1, 3)), int(g.integers(1, 4))
    n = int(g.integers(2, 10))
    T = int(g.integers(1, n + 1))
    D = int(g.integers(1, 5))
    S, R = int(g.integers(0, 4)), int(g.integers(1, 5))
    Q = g.standard_normal((Hkv * G, T, D))
    K = g.standard_normal((Hkv, n, D))
    bf = np.array(_brute_lazy(Q.tolist(), K.tolist(), G, S, R, 1 / math.sqrt(D)))
    assert np.max(np.abs(O.lazy_scores(Q, K, S, R) - bf)) < 1e-13


def test_ratio_monotone_in_window_and_sink():
    g = _rng(12)
    Q = g.standard_normal((2, 6, 8)); K = g.standard_normal((2, 80, 8))
    prev = np.zeros(2)
    for R in [1, 2, 5, 20, 79, 80, 200]:
        cur = O.lazy_scores(Q, K, 2, R)
        assert np.all(cur >= prev - 1e-15); prev = cur
    prev = np.zeros(2)
    for S in [0, 1, 2, 6, 40, 80]:
        cur = O.lazy_scores(Q, K, S, 3)
        assert np.all(cur >= prev - 1e-15); prev = cur


def test_causal_mask_inside_tail_block():
    """The tail query at position i must not see keys j > i: make the last key
    overwhelmingly attractive; only the last query may feel it."""
    D, n, T = 8, 12, 3
    Q = np.zeros((1, T, D)); Q[0, :, 0] = 1.0
    K = np.zeros((1, n, D)); K[0, n - 1, 0] = 60.0
    # S = 0, R = 1: kept set is {n-1}; rows 0,1 cannot see it -> mass 0, row 2 -> ~1
    sc = O.lazy_scores(Q, K, 0, 1, scale=1.0)
    assert abs(sc[0] - (0 + 0 + 1.0) / 3) < 1e-12


def test_tail_longer_than_window_and_no_sink():
    # T > R and S = 0: early tail rows collect nothing
    n, T, R = 10, 6, 2
    sc = O.lazy_scores(np.zeros((1, T, 4)), np.zeros((1, n, 4)), 0, R)
    exp = sum((max(0, (n - T + t) - (n - R) + 1)) / (n - T + t + 1) for t in range(T)) / T
    assert abs(sc[0] - exp) < 1e-14


# ---------------------------------------------------------------- O4 --------
@pytest.mark.parametrize("seed", range(8))
def test_select_maximises_sum_of_ratios_brute_force(seed):
    """Theorem 1: the error bound grows with sum_{i in I} s_i = sum (1 - r_i);
    the chosen set must maximise sum r over all sets of the same size."""
    g = _rng(40 + seed)
    L = int(g.integers(1, 9))
    scores = g.random((L, 2, 3))
    r = scores.reshape(L, -1).mean(axis=1)
    for n_lazy in range(L + 1):
        mask, rr = O.select_lazy(scores, n_lazy)
        assert mask.sum() == n_lazy and np.allclose(rr, r, atol=1e-15)
        best = max(sum(r[list(c)]) for c in itertools.combinations(range(L), n_lazy))
        assert abs(r[mask == 1].sum() - best) < 1e-12
        pq = O.select_lazy_priority_queue(r, L - n_lazy)
        assert np.array_equal(pq, mask)


def test_select_edges_and_ties():
    sc = np.array([0.5, 0.9, 0.5, 0.9, 0.1]).reshape(5, 1, 1)
    assert O.select_lazy(sc, 0)[0].tolist() == [0, 0, 0, 0, 0]
    assert O.select_lazy(sc, 5)[0].tolist() == [1, 1, 1, 1, 1]
    assert O.select_lazy(sc, 1)[0].tolist() == [0, 1, 0, 0, 0]      # tie -> lower index
    assert O.select_lazy(sc, 3)[0].tolist() == [1, 1, 0, 1, 0]
    for n_lazy in range(6):
        assert np.array_equal(O.select_lazy_priority_queue(sc.reshape(5), 5 - n_lazy), O.select_lazy(sc, n_lazy)[0])


def test_priority_queue_follows_figure_3_trace():
    """Hand trace of the queue of Figure 3 with P = 2 on ratios .3 .8 .5 .9 .1:
    after layer 2 arrives the queue {.3,.8,.5} overflows -> layer 1 lazy; layer 3
    (.9) is popped on arrival; layer 4 arrives -> {.3,.5,.1} overflows -> layer 2."""
    mask = O.select_lazy_priority_queue([0.3, 0.8, 0.5, 0.9, 0.1], 2)
    assert mask.tolist() == [0, 1, 1, 1, 0]


def test_priority_queue_trace_pops_on_arrival_and_ends_at_the_sorted_selection():
    """Figure 3 again, step by step: with P = 2 on .3 .8 .5 .9 .1 nothing leaves
    while layers 0, 1 arrive, layer 1 leaves when layer 2 arrives, layer 3 leaves
    on its own arrival, layer 2 leaves when layer 4 arrives."""
    mask, popped = O.select_lazy_priority_queue_trace([0.3, 0.8, 0.5, 0.9, 0.1], 2)
    assert popped.tolist() == [-1, -1, 1, 3, 2] and mask.tolist() == [0, 1, 1, 1, 0]
    g = _rng(77)
    for _ in range(20):
        L = int(g.integers(1, 12))
        r = np.round(g.random(L), 1)                     # coarse values: ties happen
        for P in range(L + 1):
            mask, popped = O.select_lazy_priority_queue_trace(r, P)
            assert np.array_equal(mask, O.select_lazy_priority_queue(r, P))
            assert np.array_equal(mask, O.select_lazy(r.reshape(L, 1, 1), L - P)[0])
            out = [x for x in popped.tolist() if x >= 0]
            assert len(out) == len(set(out)) == L - P == int(mask.sum())
            assert all(x <= l for l, x in enumerate(popped.tolist()))    # only layers that have arrived can leave
            # while at most P layers have arrived nothing leaves
            assert all(x == -1 for x in popped.tolist()[:P])


def test_per_sequence_selection_is_the_single_prompt_selection_row_by_row():
    g = _rng(78)
    L, B, Hq = 7, 4, 3
    scores = g.random((L, B, Hq))
    for n_lazy in range(L + 1):
        mask, r = O.select_lazy_per_sequence(scores, n_lazy)
        assert mask.shape == (B, L) and np.all(mask.sum(axis=1) == n_lazy)
        for b in range(B):
            rb = scores[:, b, :].mean(axis=1)
            assert np.allclose(r[b], rb, atol=1e-15)
            best = max(sum(rb[list(c)]) for c in itertools.combinations(range(L), n_lazy))
            assert abs(rb[mask[b] == 1].sum() - best) < 1e-12
    # one prompt: identical to the batch selection
    one = g.random((L, 1, Hq))
    assert np.array_equal(O.select_lazy_per_sequence(one, 3)[0][0], O.select_lazy(one, 3)[0])
    # prompts that disagree get different masks
    two = np.zeros((2, 2, 1)); two[0, 0] = 0.9; two[1, 0] = 0.1; two[0, 1] = 0.2; two[1, 1] = 0.7
    assert O.select_lazy_per_sequence(two, 1)[0].tolist() == [[1, 0], [0, 1]]


def test_frequency_selection_hand_example_and_brute_force():
    """Section 5.2: four samples over five layers; layer 3 is lazy in all four,
    layers 0 and 4 in two each, layer 1 in one, layer 2 never."""
    masks = np.array([[1, 0, 0, 1, 0],
                      [0, 1, 0, 1, 1],
                      [1, 0, 0, 1, 0],
                      [0, 0, 0, 1, 1]])
    m, c = O.select_lazy_by_frequency(masks, 2)
    assert c.tolist() == [2, 1, 0, 4, 2] and m.tolist() == [1, 0, 0, 1, 0]        # tie 0 vs 4 -> lower index
    assert O.select_lazy_by_frequency(masks, 3)[0].tolist() == [1, 0, 0, 1, 1]
    assert O.select_lazy_by_frequency(masks, 0)[0].sum() == 0 and O.select_lazy_by_frequency(masks, 5)[0].sum() == 5
    g = _rng(79)
    for _ in range(10):
        N, L = int(g.integers(1, 9)), int(g.integers(1, 8))
        mk = (g.random((N, L)) < 0.4).astype(np.uint8)
        for n_lazy in range(L + 1):
            m, c = O.select_lazy_by_frequency(mk, n_lazy)
            assert np.array_equal(c, mk.sum(axis=0)) and m.sum() == n_lazy
            best = max(sum(c[list(s_)]) for s_ in itertools.combinations(range(L), n_lazy))
            assert c[m == 1].sum() == best
    # one sample: its own mask comes back when n_lazy matches
    one = np.array([[0, 1, 1, 0]])
    assert O.select_lazy_by_frequency(one, 2)[0].tolist() == [0, 1, 1, 0]


def _brute_lazy_per_row(Q, K, G, S, R, scale):
    res = []
    for hq in range(len(Q)):
        T, n = len(Q[hq]), len(K[0])
        acc = 0.0
        for t in range(T):
            i = n - T + t
            lg = [scale * math.fsum(a * b for a, b in zip(Q[hq][t], K[hq // G][j])) for j in range(i + 1)]
            mx = max(lg)
            w = [math.exp(x - mx) for x in lg]
            acc += math.fsum(w[j] for j in range(i + 1) if (j < S or j > i - R)) / math.fsum(w)
        res.append(acc / T)
    return res


@pytest.mark.parametrize("seed", range(6))
def test_per_row_window_reading(seed):
    """Brute force; agreement with the fixed-block reading for the last query
    (T = 1); closed form for uniform attention; 1 when every row's window covers
    its keys; never below the fixed-block ratio minus the keys the block adds."""
    g = _rng(90 + seed)
    Hkv, G = int(g.integers(1, 3)), int(g.integers(1, 4))
    n = int(g.integers(2, 12))
    T = int(g.integers(1, n + 1))
    D = int(g.integers(1, 5))
    S, R = int(g.integers(0, 4)), int(g.integers(1, 6))
    Q = g.standard_normal((Hkv * G, T, D))
    K = g.standard_normal((Hkv, n, D))
    got = O.lazy_scores_per_row_window(Q, K, S, R)
    bf = np.array(_brute_lazy_per_row(Q.tolist(), K.tolist(), G, S, R, 1 / math.sqrt(D)))
    assert np.max(np.abs(got - bf)) < 1e-13
    last = O.lazy_scores_per_row_window(Q[:, -1:], K, S, R)
    assert np.max(np.abs(last - O.lazy_scores(Q[:, -1:], K, S, R))) < 1e-13
    z = O.lazy_scores_per_row_window(np.zeros((1, T, D)), K[:1], S, R)[0]
    exp = sum(len({j for j in range(i + 1) if j < S or j > i - R}) / (i + 1) for i in range(n - T, n)) / T
    assert abs(z - exp) < 1e-13
    assert np.max(np.abs(O.lazy_scores_per_row_window(Q, K, S, n) - 1.0)) < 1e-12


# ---------------------------------------------------------------- O5 --------
@pytest.mark.parametrize("S,R", [(0, 1), (0, 5), (4, 1), (4, 6), (3, 8), (2, 2)])
def test_ring_exhaustive(S, R):
    C = S + R
    for n in range(0, 4 * C + 3):
        # brute-force replay of which token sits where
        sim = [None] * C
        for p in range(n):
            sim[O.ring_slot(p, S, R)] = p
        for s in range(C):
            assert O.ring_owner(s, n, S, R) == sim[s]
        held = sorted(p for p in sim if p is not None)
        expect = sorted(set(range(min(S, n))) | set(range(max(S, n - R), n)))
        assert held == expect                      # exactly sinks + last R non-sink tokens
        assert len(held) == O.ring_valid_slots(n, S, R)
        # valid slots are the contiguous prefix of the cache
        assert [s for s in range(C) if sim[s] is not None] == list(range(len(held)))
    # identity placement before the first wrap
    assert all(O.ring_slot(p, S, R) == p for p in range(C))
    # sinks are never overwritten
    assert all(O.ring_slot(p, S, R) >= S for p in range(S, 5 * C))
    # any R consecutive non-sink positions map to R distinct slots
    for p0 in range(S, S + 3 * R):
        assert len({O.ring_slot(p, S, R) for p in range(p0, p0 + R)}) == R


def test_stream_cache_after_holds_owner_bits():
    S, R = 2, 5
    hist = np.arange(23 * 3, dtype=np.int32).reshape(23, 3)
    cache, valid = O.stream_cache_after(hist, S, R)
    assert valid == 7
    for s in range(S + R):
        assert np.array_equal(cache[s], hist[O.ring_owner(s, 23, S, R)])
    cache2, valid2 = O.stream_cache_after(hist[:4], S, R)
    assert valid2 == 4 and np.array_equal(cache2[:4], hist[:4]) and not cache2[4:].any()


def test_streaming_attention_on_ring_contents_equals_logical_history():
    """Attention over the rows the ring holds (any order) equals O2 on the
    complete history: the ring keeps exactly the kept set."""
    g = _rng(50)
    S, R, n, D = 3, 6, 40, 8
    q = g.standard_normal((2, D)); K = g.standard_normal((1, n, D)); V = g.standard_normal((1, n, D))
    ck, valid = O.stream_cache_after(K[0], S, R)
    cv, _ = O.stream_cache_after(V[0], S, R)
    a = O.full_attention(q, ck[None, :valid], cv[None, :valid])
    b = O.streaming_attention(q, K, V, S, R)
    assert np.max(np.abs(a - b)) < 1e-13


def test_hybrid_replay_sequence():
    g = _rng(51)
    S, R, D = 2, 4, 8
    rp = O.HybridReplay([0, 1], S, R)
    K0 = g.standard_normal((1, 5, D)); V0 = g.standard_normal((1, 5, D))
    for l in range(2):
        rp.load_prompt(l, K0, V0)
    for step in range(6):
        k = g.standard_normal((1, D)); v = g.standard_normal((1, D)); q = g.standard_normal((2, D))
        for l in range(2):
            rp.append(l, k, v)
        n = 5 + step + 1
        assert rp.K[0].shape[1] == n
        full = rp.attend(0, q); lazy = rp.attend(1, q)
        assert np.allclose(full, O.full_attention(q, rp.K[0], rp.V[0]))
        assert np.allclose(lazy, O.streaming_attention(q, rp.K[1], rp.V[1], S, R))
        assert np.allclose(full, lazy) == (n <= S + R)
