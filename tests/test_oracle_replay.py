"""Pins of the replay-visibility oracle (paper Appendix A.3 and the replay-mask figure of
Section 4.5): the figure's printed example, a token-by-token simulation of the cache with Python
sets, block-level units with a short last unit, and the steady-state alive-set size of the
proposition in Appendix A.2."""
import json
import os

import numpy as np

from oracle import replay

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "replay_mask_figure.json")


def units_from_evicted(alive, evicted):
    """Ascending compacted indices of the entries of `alive` that are not evicted (block = 1)."""
    return [i for i, t in enumerate(alive) if t not in evicted]


def test_figure_example_rows_and_survivors():
    g = json.load(open(GOLDEN))
    T = g["tokens"]
    total_before = [r["after_token"] + 1 for r in g["rounds"]]                   # [5, 8]
    alive = list(range(total_before[0]))                                         # A_0 = block_0
    kept_lists, alive_before = [], []
    for i, r in enumerate(g["rounds"]):
        alive_before.append(len(alive))
        kept_lists.append(units_from_evicted(alive, set(r["evicts"])))
        alive = [alive[j] for j in kept_lists[-1]]
        if i + 1 < len(total_before):
            alive += list(range(total_before[i], total_before[i + 1]))          # block_{r+1}
    k_max = max(len(k) for k in kept_lists)
    ks = np.full((2, 1, 1, k_max), -1, np.int32)
    for r, k in enumerate(kept_lists):
        ks[r, 0, 0, : len(k)] = k
    pos, count, rc = replay.alive_positions(ks, [[len(k)] for k in kept_lists], [[a] for a in alive_before],
                                            [[t] for t in total_before])
    assert rc == 0
    assert list(pos[0, 0, 0, : count[0, 0, 0]]) == [0, 2, 4]                     # round 1 evicts t1, t3
    assert list(pos[1, 0, 0, : count[1, 0, 0]]) == g["final_survivors"]          # round 2 evicts t2, t5
    M = replay.dense_mask(T, total_before, [pos[r, 0, 0, : count[r, 0, 0]] for r in range(2)])
    for row, vis in g["visible"].items():
        assert list(np.nonzero(M[int(row)])[0]) == vis
    for t in range(total_before[0]):                                             # before the first round: plain causal
        assert list(np.nonzero(M[t])[0]) == list(range(t + 1))


def simulate_with_sets(T, boundaries, decisions):
    """Token-by-token cache simulation: visible[t] = the alive set when token t is generated (itself
    included); at a boundary the decision (set of evicted original positions) is applied."""
    alive, vis = set(), []
    for t in range(T):
        alive.add(t)
        vis.append(set(alive))
        if t + 1 in boundaries:
            alive -= decisions[boundaries.index(t + 1)]
    return vis


def test_dense_mask_equals_set_simulation_random_blocks():
    rng = np.random.default_rng(3)
    for trial in range(20):
        block = int(rng.choice([1, 1, 2, 4]))
        R = int(rng.integers(1, 5))
        grows = [int(rng.integers(2, 9)) for _ in range(R + 1)]
        boundaries = list(np.cumsum(grows[:-1]))
        T = int(sum(grows))
        alive, kept_lists, alive_before, evicted_sets = list(range(grows[0])), [], [], []
        for r in range(R):
            n_units = (len(alive) + block - 1) // block
            K = int(rng.integers(0, n_units + 1))
            units = sorted(rng.choice(n_units, K, replace=False).tolist())
            keep_idx = [i for u in units for i in range(u * block, min((u + 1) * block, len(alive)))]
            alive_before.append(len(alive))
            kept_lists.append(units)
            evicted_sets.append(set(alive) - {alive[i] for i in keep_idx})
            alive = [alive[i] for i in keep_idx] + list(range(boundaries[r], boundaries[r] + grows[r + 1]))
        k_max = max(1, max(len(k) for k in kept_lists))
        ks = np.full((R, 1, 1, k_max), -1, np.int32)
        for r, k in enumerate(kept_lists):
            ks[r, 0, 0, : len(k)] = k
        pos, count, rc = replay.alive_positions(ks, [[len(k)] for k in kept_lists], [[a] for a in alive_before],
                                                [[int(t)] for t in boundaries], block)
        assert rc == 0
        M = replay.dense_mask(T, boundaries, [pos[r, 0, 0, : count[r, 0, 0]] for r in range(R)])
        vis = simulate_with_sets(T, [int(x) for x in boundaries], evicted_sets)
        for t in range(T):
            assert set(np.nonzero(M[t])[0].tolist()) == vis[t], (trial, t)


def test_steady_state_alive_size_and_error_codes():
    # delta = 512 new tokens per round, keep one third of 768: the alive set returns to delta / epsilon = 768
    R, delta, K = 5, 512, 256
    rng = np.random.default_rng(1)
    ks = np.stack([np.sort(rng.choice(768, K, replace=False)) for _ in range(R)]).astype(np.int32).reshape(R, 1, 1, K)
    pos, count, rc = replay.alive_positions(ks, np.full((R, 1), K), np.full((R, 1), 768), [[768 + r * delta] for r in range(R)])
    assert rc == 0 and np.all(count == K)
    for r in range(R):
        p = pos[r, 0, 0]
        assert np.all(np.diff(p) > 0) and p.max() < 768 + r * delta
        if r:
            assert np.sum(p >= 768 + (r - 1) * delta) == np.sum(ks[r, 0, 0] >= K)     # survivors of the newest block
    bad = ks.copy()
    bad[2, 0, 0, 5] = bad[2, 0, 0, 4]
    _, c2, rc = replay.alive_positions(bad, np.full((R, 1), K), np.full((R, 1), 768), [[768 + r * delta] for r in range(R)])
    assert rc == 3 and np.all(c2[:2] == K) and np.all(c2[2:] == -1)
    fewer = np.full((R, 1), 768)
    fewer[1] = 100                      # fewer tokens alive at round 1 than round 0 kept
    _, _, rc = replay.alive_positions(ks, np.full((R, 1), K), fewer, [[768 + r * delta] for r in range(R)])
    assert rc == 1


def test_replay_attention_pins():
    """Causal mask -> the library's scaled_dot_product_attention; and the paper's claim itself: under the
    replay mask, token t's attention equals decode attention over the cache as it stood at rollout time
    (two separately written oracle routines: dense numpy here, the C++ ragged decode + compaction there)."""
    import torch
    import oracle
    rng = np.random.default_rng(0)
    q, k, v = rng.normal(size=(4, 9, 8)), rng.normal(size=(2, 9, 8)), rng.normal(size=(2, 9, 8))
    o = replay.replay_attention(q, k, v, np.tril(np.ones((9, 9), bool))[None])
    ref = torch.nn.functional.scaled_dot_product_attention(torch.tensor(q)[None], torch.tensor(k).repeat_interleave(2, 0)[None],
                                                           torch.tensor(v).repeat_interleave(2, 0)[None], is_causal=True)[0].numpy()
    assert np.abs(o - ref).max() < 1e-12
    # rollout: 1 layer, prompt of 6 tokens, rounds after 6 and 11 tokens keep 3 of 6 and 4 of 8 cache entries
    L, B, Hq, Hkv, d, T = 1, 1, 4, 2, 64, 15
    kf = rng.normal(size=(L, Hkv, T, d)).astype(np.float32)
    vf = rng.normal(size=(L, Hkv, T, d)).astype(np.float32)
    qf = rng.normal(size=(L, B, Hq, T, d)).astype(np.float32)
    total_before, kept_lists = [6, 11], [[0, 2, 5], [1, 2, 4, 7]]
    cache_k = np.zeros((L, Hkv, T, d), np.float32)
    cache_v = np.zeros_like(cache_k)
    so, lens = np.array([0, T], np.int64), np.zeros(1, np.int32)
    rollout_out = np.zeros((Hq, T, d))
    r = 0
    for t in range(T):
        out, rc = oracle.decode_attn(cache_k, cache_v, so, lens, qf[:, :, :, t], kf[:, None, :, t].copy(), vf[:, None, :, t].copy())
        assert rc == 0
        rollout_out[:, t] = out[0, 0]
        if r < 2 and t + 1 == total_before[r]:
            ks = np.array(kept_lists[r], np.int32)[None, None]
            cache_k, cache_v, nl, rc = oracle.compact_kv(cache_k, cache_v, so, lens, ks, [len(kept_lists[r])], 0)
            assert rc == 0
            lens = nl.copy()
            r += 1
    k_max = 4
    ks = np.full((2, 1, 1, k_max), -1, np.int32)
    ks[0, 0, 0, :3], ks[1, 0, 0, :4] = kept_lists[0], kept_lists[1]
    pos, cnt, rc = replay.alive_positions(ks, [[3], [4]], [[6], [8]], [[6], [11]])
    assert rc == 0
    M = replay.dense_mask(T, total_before, [pos[i, 0, 0, : cnt[i, 0, 0]] for i in range(2)])
    rep = replay.replay_attention(qf[0, 0].astype(np.float64), kf[0].astype(np.float64), vf[0].astype(np.float64), M[None])
    assert np.abs(rep - rollout_out).max() < 1e-10


def _random_list_history(rng, R, block, boundaries, grows):
    """One list's rollout: random unit decisions at every boundary.  Returns the kept units per round, the alive
    count when each round fired, and the evicted ORIGINAL positions per round (for the set simulation)."""
    alive, kept_lists, alive_before, evicted_sets = list(range(grows[0])), [], [], []
    for r in range(R):
        n_units = (len(alive) + block - 1) // block
        K = int(rng.integers(1, n_units + 1))
        units = sorted(rng.choice(n_units, K, replace=False).tolist())
        keep_idx = [i for u in units for i in range(u * block, min((u + 1) * block, len(alive)))]
        alive_before.append(len(alive))
        kept_lists.append(units)
        evicted_sets.append(set(alive) - {alive[i] for i in keep_idx})
        alive = [alive[i] for i in keep_idx] + list(range(boundaries[r], boundaries[r] + grows[r + 1]))
    return kept_lists, alive_before, evicted_sets


def test_per_list_alive_counts_match_independent_lists_and_set_simulation():
    """Several lists per sequence whose alive counts differ (Section 4.1: every layer evicts the same fraction but not
    the same entries, so with units of several tokens a short last unit kept by one layer and evicted by another
    leaves the layers with different lengths).  The [R][B][G] form of `alive_before` must give, list by list, what G
    separate single-list calls give, and each list must agree with the token-by-token set simulation."""
    rng = np.random.default_rng(11)
    for trial in range(12):
        block = int(rng.choice([4, 32]))
        R, B, G = int(rng.integers(2, 5)), 2, 3
        # growth that is NOT a multiple of the unit, so that the last unit of a round is short
        grows = [[int(rng.integers(block + 1, 3 * block + 2)) | 1 for _ in range(R + 1)] for _ in range(B)]
        hist = [[None] * G for _ in range(B)]
        bounds = [[int(x) for x in np.cumsum(grows[b][:-1])] for b in range(B)]
        # every list of a sequence keeps the same number of UNITS per round (one budget per sequence), drawn per
        # sequence; which units -- and therefore whether the short last one survives -- differs per list
        for b in range(B):
            alive = [list(range(grows[b][0])) for _ in range(G)]
            kept_l = [[] for _ in range(G)]
            ab_l = [[] for _ in range(G)]
            ev_l = [[] for _ in range(G)]
            for r in range(R):
                n_units = [(len(a) + block - 1) // block for a in alive]
                K = int(rng.integers(1, min(n_units) + 1))
                for g in range(G):
                    units = sorted(rng.choice(n_units[g], K, replace=False).tolist())
                    if g == 0 and n_units[g] - 1 not in units:          # list 0 always keeps the (short) last unit
                        units[-1] = n_units[g] - 1
                    if g == 1 and K < n_units[g] and n_units[g] - 1 in units:   # list 1 drops it when it can
                        free = sorted(set(range(n_units[g] - 1)) - set(units))
                        units = sorted(units[:-1] + [free[0]])
                    keep_idx = [i for u in units for i in range(u * block, min((u + 1) * block, len(alive[g])))]
                    ab_l[g].append(len(alive[g]))
                    kept_l[g].append(units)
                    ev_l[g].append(set(alive[g]) - {alive[g][i] for i in keep_idx})
                    alive[g] = [alive[g][i] for i in keep_idx] + list(range(bounds[b][r], bounds[b][r] + grows[b][r + 1]))
            for g in range(G):
                hist[b][g] = (kept_l[g], ab_l[g], ev_l[g])
        k_max = max(len(k) for b in range(B) for g in range(G) for k in hist[b][g][0])
        ks = np.full((R, B, G, k_max), -1, np.int32)
        budget = np.zeros((R, B), np.int32)
        ab = np.zeros((R, B, G), np.int32)
        tb = np.zeros((R, B), np.int32)
        for b in range(B):
            for g in range(G):
                for r in range(R):
                    u = hist[b][g][0][r]
                    ks[r, b, g, : len(u)] = u
                    budget[r, b] = len(u)
                    ab[r, b, g] = hist[b][g][1][r]
                    tb[r, b] = bounds[b][r]
        assert any(len(set(ab[r, b])) > 1 for r in range(R) for b in range(B)), "the lists never disagreed"
        pos, count, rc = replay.alive_positions(ks, budget, ab, tb, block)
        assert rc == 0
        for b in range(B):
            T = int(sum(grows[b]))
            for g in range(G):
                # (i) the per-list call equals a single-list call on that list alone
                p1, c1, rc1 = replay.alive_positions(ks[:, b:b + 1, g:g + 1], budget[:, b:b + 1], ab[:, b:b + 1, g],
                                                     tb[:, b:b + 1], block)
                assert rc1 == 0
                assert np.array_equal(c1[:, 0, 0], count[:, b, g])
                assert np.array_equal(p1[:, 0, 0], pos[:, b, g])
                # (ii) and the token-by-token simulation of that list's cache
                M = replay.dense_mask(T, bounds[b], [pos[r, b, g, : count[r, b, g]] for r in range(R)])
                vis = simulate_with_sets(T, bounds[b], hist[b][g][2])
                for t in range(T):
                    assert set(np.nonzero(M[t])[0].tolist()) == vis[t], (trial, b, g, t)


def test_per_list_form_is_not_confused_with_the_per_sequence_form():
    """[R][B] alive counts are broadcast over the lists; [R][B][G] counts are taken list by list in that index order
    (a transposed reshape would hand list g of sequence b the count of another list)."""
    R, B, G, block = 1, 2, 2, 1
    ks = np.full((R, B, G, 3), -1, np.int32)
    ab = np.array([[[3, 5], [4, 6]]], np.int32)                  # [R][B][G]: all different
    for b in range(B):
        for g in range(G):
            ks[0, b, g, :2] = [0, ab[0, b, g] - 1]               # keep the first and the last alive entry
    tb = np.full((R, B), 6, np.int32)
    pos, count, rc = replay.alive_positions(ks, np.full((R, B), 2), ab, tb, block)
    assert rc == 0 and np.all(count == 2)
    for b in range(B):
        for g in range(G):
            n = int(ab[0, b, g])                                 # A_0 = the last n positions before 6
            assert list(pos[0, b, g, :2]) == [6 - n, 5]
    # broadcast form: one count per sequence
    pos2, count2, rc = replay.alive_positions(ks[:, :, :1], np.full((R, B), 2), ab[:, :, 0], tb, block)
    assert rc == 0 and list(pos2[0, 1, 0, :2]) == [6 - 4, 5]
