"""Pins for the oracle's Gumbel-top-k sampler (Section 4.3) and Eq. (1).

* brute force: every ordered keep-tuple of a tiny list is enumerated and its
  Plackett-Luce probability computed here with plain Python arithmetic; the
  oracle's Eq. (1) must reproduce each one, they must sum to 1, and the
  oracle's sampler must draw tuples (and sets) with those frequencies;
* closed forms / textbook cases for Eq. (1);
* invariants of the sampler; greedy mode against a library sort.
"""
import itertools
import math

import numpy as np
import pytest
from scipy.special import log_softmax, logsumexp
from scipy.stats import chi2

import oracle


def pl_tuple_prob(s, sigma, cand):
    """Sequential sampling without replacement with probabilities proportional to exp(s)."""
    rem = list(cand)
    p = 1.0
    for t in sigma:
        z = sum(math.exp(s[i]) for i in rem)
        p *= math.exp(s[t]) / z
        rem.remove(t)
    return p


def all_tuples(cand, k):
    return list(itertools.permutations(cand, k))


# ---------------------------------------------------------------- Eq. (1)

@pytest.mark.parametrize("N,P,K", [(5, 0, 2), (6, 0, 3), (6, 2, 4), (4, 0, 4), (7, 1, 2)])
def test_logprob_brute_force_enumeration(N, P, K):
    rng = np.random.default_rng(N * 100 + P * 10 + K)
    s = rng.normal(0, 1.5, N).astype(np.float32)
    cand = list(range(P, N))
    tuples = all_tuples(cand, K - P)
    ko = np.array(tuples, np.int32).reshape(len(tuples), 1, K - P) if K > P else np.zeros((1, 1, 1), np.int32)
    B = len(tuples)
    logits = np.broadcast_to(s, (B, 1, N))
    lp, rc = oracle.evict_logprob(logits, [N] * B, [P] * B, [K] * B, ko)
    assert rc == 0
    lp = lp.reshape(-1)
    want = np.array([pl_tuple_prob([float(x) for x in s], t, cand) for t in tuples])
    assert np.allclose(np.exp(lp), want, rtol=1e-12, atol=0)
    assert abs(np.exp(lp).sum() - 1.0) < 1e-12
    lp2, _ = oracle.evict_logprob_scan(logits, [N] * B, [P] * B, [K] * B, ko)
    assert np.allclose(lp2.reshape(-1), lp, rtol=0, atol=1e-12)


def test_logprob_hand_example():
    # exp(s) = 1, 2, 3; sigma = (2, 0): 3/6 * 1/3 = 1/6
    s = np.log(np.array([1.0, 2.0, 3.0])).astype(np.float32)
    lp, _ = oracle.evict_logprob(s.reshape(1, 1, 3), [3], [0], [2], np.array([[[2, 0]]], np.int32))
    assert abs(lp.item() - math.log(1.0 / 6.0)) < 2e-7
    # sigma = (1, 2, 0): 2/6 * 3/4 * 1 = 1/4
    lp, _ = oracle.evict_logprob(s.reshape(1, 1, 3), [3], [0], [3], np.array([[[1, 2, 0]]], np.int32))
    assert abs(lp.item() - math.log(0.25)) < 2e-7


def test_logprob_single_draw_is_log_softmax():
    rng = np.random.default_rng(5)
    N = 300
    s = rng.normal(0, 2, N).astype(np.float32)
    ref = log_softmax(s.astype(np.float64))
    for t in (0, 17, N - 1):
        lp, _ = oracle.evict_logprob(s.reshape(1, 1, N), [N], [0], [1], np.array([[[t]]], np.int32))
        assert abs(lp.item() - ref[t]) < 1e-12


def test_logprob_constant_logits_closed_form():
    for N, P, K in [(50, 0, 20), (64, 8, 40), (33, 0, 33)]:
        s = np.full(N, 0.7, np.float32)
        sigma = np.random.default_rng(N).permutation(np.arange(P, N))[:K - P].astype(np.int32)
        want = -sum(math.log(N - P - j) for j in range(K - P))
        for fn in (oracle.evict_logprob, oracle.evict_logprob_scan):
            lp, _ = fn(s.reshape(1, 1, N), [N], [P], [K], sigma.reshape(1, 1, -1))
            assert abs(lp.item() - want) < 1e-10


def test_logprob_full_permutation_and_shift_invariance_and_protected_ignored():
    rng = np.random.default_rng(9)
    N, P = 40, 5
    s = rng.normal(0, 3, N).astype(np.float32)
    sigma = rng.permutation(np.arange(P, N)).astype(np.int32)
    s64 = s.astype(np.float64)
    # Plackett-Luce of a full ranking: sum_j s_sigma_j - logsumexp(s over sigma_j..sigma_end)
    want = sum(s64[sigma[j]] - logsumexp(s64[sigma[j:]]) for j in range(N - P))
    lp, _ = oracle.evict_logprob(s.reshape(1, 1, N), [N], [P], [N], sigma.reshape(1, 1, -1))
    assert abs(lp.item() - want) < 1e-9
    lp_scan, _ = oracle.evict_logprob_scan(s.reshape(1, 1, N), [N], [P], [N], sigma.reshape(1, 1, -1))
    assert abs(lp_scan.item() - want) < 1e-9
    # adding a constant to every logit changes nothing (exactly representable shift)
    lp_shift, _ = oracle.evict_logprob((s + np.float32(4.0)).reshape(1, 1, N), [N], [P], [N], sigma.reshape(1, 1, -1))
    assert abs(lp_shift.item() - want) < 1e-4
    # protected units are not part of the choice
    s2 = s.copy()
    s2[:P] = 50.0
    lp_p, _ = oracle.evict_logprob(s2.reshape(1, 1, N), [N], [P], [N], sigma.reshape(1, 1, -1))
    assert lp_p.item() == lp.item()


def test_logprob_scan_equals_literal_medium_and_extreme():
    rng = np.random.default_rng(11)
    N, K = 700, 650      # little mass remains at the end: the subtractive prefix form would cancel
    s = rng.normal(0, 4, (3, 2, N)).astype(np.float32)
    ko, _, _, st = oracle.sample_evict(s, [N] * 3, None, [K] * 3, K, seed=3, rnd=0)
    assert not st.any()
    a, _ = oracle.evict_logprob(s, [N] * 3, None, [K] * 3, ko)
    b, _ = oracle.evict_logprob_scan(s, [N] * 3, None, [K] * 3, ko)
    assert np.allclose(a, b, rtol=0, atol=1e-8)
    assert np.all(a < 0)


def test_logprob_rejects_bad_sigma():
    s = np.zeros((1, 1, 6), np.float32)
    for sig in ([1, 1], [0, 9], [0, -1]):
        lp, rc = oracle.evict_logprob(s, [6], [0], [2], np.array([[sig]], np.int32))
        assert rc == 3 and math.isnan(lp.item())
    lp, rc = oracle.evict_logprob(s, [6], [3], [2], np.array([[[4, 5]]], np.int32))
    assert rc == 1


# ---------------------------------------------------------------- sampler

@pytest.mark.parametrize("N,P,K,greedy", [(5, 0, 2, 0), (6, 1, 3, 0), (5, 0, 5, 0)])
def test_sampler_frequencies_match_enumeration(N, P, K, greedy):
    """Gumbel-top-k == sequential sampling without replacement (chi-square, tuples and sets)."""
    rng = np.random.default_rng(N + K)
    s = rng.normal(0, 1.0, N).astype(np.float32)
    draws = 300000
    logits = np.broadcast_to(s, (draws, 1, N))
    ko, ks, km, st = oracle.sample_evict(logits, [N] * draws, [P] * draws, [K] * draws, K, seed=12345, rnd=7)
    assert not st.any()
    cand = list(range(P, N))
    tuples = all_tuples(cand, K - P)
    probs = np.array([pl_tuple_prob([float(x) for x in s], t, cand) for t in tuples])
    assert abs(probs.sum() - 1) < 1e-12
    index = {t: i for i, t in enumerate(tuples)}
    counts = np.zeros(len(tuples))
    for row in ko[:, 0, :K - P]:
        counts[index[tuple(int(x) for x in row)]] += 1
    stat = ((counts - draws * probs) ** 2 / (draws * probs)).sum()
    assert stat < chi2.ppf(0.9999, len(tuples) - 1), stat
    # sets: probability = sum over the orders
    set_p = {}
    set_c = {}
    for t, p, c in zip(tuples, probs, counts):
        key = tuple(sorted(t))
        set_p[key] = set_p.get(key, 0) + p
        set_c[key] = set_c.get(key, 0) + c
    if len(set_p) > 1:
        sp = np.array(list(set_p.values()))
        sc = np.array(list(set_c.values()))
        stat = ((sc - draws * sp) ** 2 / (draws * sp)).sum()
        assert stat < chi2.ppf(0.9999, len(sp) - 1)


def test_sampler_rounds_and_lists_are_independent_streams():
    s = np.zeros((4, 3, 64), np.float32)
    a = oracle.sample_evict(s, [64] * 4, None, [16] * 4, 16, seed=1, rnd=0)[0]
    b = oracle.sample_evict(s, [64] * 4, None, [16] * 4, 16, seed=1, rnd=1)[0]
    c = oracle.sample_evict(s, [64] * 4, None, [16] * 4, 16, seed=2, rnd=0)[0]
    assert not np.array_equal(a, b) and not np.array_equal(a, c)
    flat = a.reshape(12, 16)
    assert len({tuple(r) for r in flat}) == 12       # every list has its own noise
    # list_base shifts the stream: lists 2.. of a base-0 call == lists 0.. of a base-6 call
    d = oracle.sample_evict(s[2:], [64] * 2, None, [16] * 2, 16, seed=1, rnd=0, list_base=6)[0]
    assert np.array_equal(d, a[2:])


def test_sampler_invariants_random_shapes():
    rng = np.random.default_rng(21)
    for trial in range(30):
        B, G = int(rng.integers(1, 5)), int(rng.integers(1, 4))
        n_max = int(rng.integers(1, 200))
        n = rng.integers(0, n_max + 1, B).astype(np.int32)
        P = np.array([rng.integers(0, x + 1) for x in n], np.int32)
        K = np.array([rng.integers(p, x + 1) for p, x in zip(P, n)], np.int32)
        k_max = max(int(K.max()), 1)
        s = rng.normal(0, 1, (B, G, n_max)).astype(np.float32)
        ko, ks, km, st = oracle.sample_evict(s, n, P, K, k_max, seed=trial, rnd=trial)
        assert not st.any()
        for b in range(B):
            for g in range(G):
                kept = ks[b, g, :K[b]]
                assert np.all(ks[b, g, K[b]:] == -1) and np.all(ko[b, g, K[b] - P[b]:] == -1)
                assert np.all(np.diff(kept) > 0) and (K[b] == 0 or (kept[0] >= 0 and kept[-1] < n[b]))
                assert np.array_equal(kept[:P[b]], np.arange(P[b]))          # protected prefix kept
                assert km[b, g].sum() == K[b] and np.all(km[b, g, kept] == 1)
                order = ko[b, g, :K[b] - P[b]]
                assert sorted(order.tolist()) == kept[P[b]:].tolist()
                keys = [oracle.perturbed_key(float(s[b, g, i]), trial, trial, b * G + g, int(i)) for i in order]
                assert all(keys[i] >= keys[i + 1] for i in range(len(keys) - 1))
                if K[b] - P[b] > 0 and K[b] < n[b]:
                    rest = [i for i in range(P[b], n[b]) if km[b, g, i] == 0]
                    worst_kept = keys[-1]
                    best_rest = max(oracle.perturbed_key(float(s[b, g, i]), trial, trial, b * G + g, i) for i in rest)
                    assert best_rest <= worst_kept


def test_greedy_equals_library_sort_with_index_tiebreak():
    rng = np.random.default_rng(4)
    N, K = 500, 123
    s = rng.integers(-3, 4, (2, 2, N)).astype(np.float32)     # many exact ties
    ko, ks, km, st = oracle.sample_evict(s, [N, N], None, [K, K], K, seed=0, rnd=0, greedy=1)
    for b in range(2):
        for g in range(2):
            ref = np.lexsort((np.arange(N), -s[b, g].astype(np.float64)))[:K]     # key desc, index asc
            assert np.array_equal(ko[b, g], ref)
            assert np.array_equal(ks[b, g], np.sort(ref))


def test_sampler_infinities_and_status():
    s = np.zeros((1, 1, 8), np.float32)
    s[0, 0, 3] = np.inf
    s[0, 0, 5] = -np.inf
    ko, ks, km, st = oracle.sample_evict(s, [8], None, [7], 7, seed=5, rnd=5)
    assert ko[0, 0, 0] == 3 and km[0, 0, 5] == 0 and st[0, 0] == 0      # -inf is never chosen ...
    ko, ks, km, st = oracle.sample_evict(s, [8], None, [8], 8, seed=5, rnd=5)
    assert ko[0, 0, 0] == 3 and ko[0, 0, 7] == 5 and st[0, 0] == 0      # ... unless forced by the count
    s[0, 0, 1] = np.nan
    ko, ks, km, st = oracle.sample_evict(s, [8], None, [7], 7, seed=5, rnd=5)
    assert st[0, 0] == 2 and np.all(ko == -1) and np.all(ks == -1) and km.sum() == 0
    s[0, 0, 1] = 0
    for n, P, K in [(8, 5, 4), (8, 0, 9), (9, 0, 2)]:
        st = oracle.sample_evict(s, [n], [P], [K], 7, seed=5, rnd=5)[3]
        assert st[0, 0] == 1
    # NaN among protected units is not looked at
    s[0, 0, 0] = np.nan
    st = oracle.sample_evict(s, [8], [2], [4], 7, seed=5, rnd=5)[3]
    assert st[0, 0] == 0


# ------------------------------------------------------------------ gradient of Eq. (1)

def test_logprob_grad_matches_finite_differences_of_eq1():
    """The gradient routine against central differences of the (independently pinned) literal Eq. (1)."""
    rng = np.random.default_rng(5)
    B, G, n_max = 2, 2, 9
    logits = rng.normal(0, 1.2, (B, G, n_max)).astype(np.float32)
    n = np.array([9, 7], np.int32)
    P = np.array([1, 0], np.int32)
    K = np.array([5, 3], np.int32)
    ko = oracle.sample_evict(logits, n, P, K, 5, seed=2, rnd=0)[0]
    grad, rc = oracle.evict_logprob_grad(logits, n, P, K, ko)
    assert rc == 0
    h = 2.0 ** -7
    for b in range(B):
        for g in range(G):
            for t in range(n_max):
                up, dn = logits.copy(), logits.copy()
                up[b, g, t] += h
                dn[b, g, t] -= h
                fd = (oracle.evict_logprob(up, n, P, K, ko)[0][0, b, g] - oracle.evict_logprob(dn, n, P, K, ko)[0][0, b, g]) / \
                     (float(up[b, g, t]) - float(dn[b, g, t]))
                want = fd if P[b] <= t < n[b] else 0.0
                assert abs(grad[0, b, g, t] - want) < 2e-4, (b, g, t)


def test_logprob_grad_closed_forms_and_invariants():
    from scipy.special import softmax
    rng = np.random.default_rng(6)
    n_max = 12
    logits = rng.normal(0, 1, (3, 1, n_max)).astype(np.float32)
    n = np.array([12, 10, 12], np.int32)
    P = np.array([0, 2, 0], np.int32)
    K = np.array([1, 6, 12], np.int32)
    ko = oracle.sample_evict(logits, n, P, K, 12, seed=4, rnd=1)[0]
    grad, rc = oracle.evict_logprob_grad(logits, n, P, K, ko)
    assert rc == 0
    # one draw: one-hot minus softmax (textbook)
    want = -softmax(logits[0, 0].astype(np.float64))
    want[ko[0, 0, 0]] += 1.0
    assert np.allclose(grad[0, 0, 0], want, atol=1e-12)
    # Eq. (1) is invariant to a common shift of the logits: the gradient sums to zero; protected units get none
    assert np.allclose(grad[0, :, 0].sum(-1), 0.0, atol=1e-12)
    assert np.all(grad[0, 1, 0, :2] == 0.0) and np.all(grad[0, 1, 0, 10:] == 0.0)
    # constant logits: drawn at step m -> 1 - sum_{j<=m} 1/(N-j+1); never drawn -> -sum_{j<=K} 1/(N-j+1)
    const = np.full((1, 1, 10), 0.7, np.float32)
    order = np.array([[[3, 9, 0, 5]]], np.int32)
    g2, rc = oracle.evict_logprob_grad(const, [10], None, [4], order)
    H = np.cumsum(1.0 / (10 - np.arange(4)))
    want = np.full(10, -H[3])
    for m, t in enumerate(order[0, 0]):
        want[t] = 1.0 - H[m]
    assert rc == 0 and np.allclose(g2[0, 0, 0], want, atol=1e-12)
    # upstream gradient scales the list; invalid list -> NaN
    g3, _ = oracle.evict_logprob_grad(const, [10], None, [4], order, grad_logp=np.array([[[-2.5]]]))
    assert np.allclose(g3, -2.5 * g2)
    bad = order.copy()
    bad[0, 0, 1] = 3
    g4, rc = oracle.evict_logprob_grad(const, [10], None, [4], bad)
    assert rc == 3 and np.isnan(g4).all()
