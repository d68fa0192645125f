"""CPU oracle for the replay visibility of Neural Garbage Collection (paper Appendix A.3,
"Reconstructing Replay Attention Masks from Retention Decisions", and the replay-mask figure
of Section 4.5).

TEST INFRASTRUCTURE ONLY: plain numpy and Python loops, written to be checked against the
paper by eye.  It shares nothing with the CUDA library and must never be called from the
product path.

The paper's construction, in its notation: the sequence is cut into blocks at the eviction
rounds; the alive set starts as A_0 = block_0; applying the retention decision d_r to A_r
gives kept_r = {i in A_r : d_{r,i} = 1}; the next alive set is A_{r+1} = kept_r U block_{r+1};
a query in block r+1 sees every token of kept_r plus, causally, the tokens of its own block;
the diagonal is set to 1.

Retention decisions arrive the way the library stores them: for round r the ascending list of
kept UNITS (`kept_sorted`), a unit being `block` consecutive entries of A_r in its current
order (the last unit may be short).  Pins (tests/test_oracle_replay.py): the figure's worked
example, a token-by-token simulation of the cache written with Python sets, and the
steady-state size of the alive set.
"""
from __future__ import annotations

import numpy as np


def alive_positions(kept_sorted, budget, alive_before, total_before, block=1):
    """kept_r in ORIGINAL token positions, for every round and list.

    kept_sorted  [R][B][G][k_max] int32  kept units of round r, ascending, -1 padded
    budget       [R][B]           int32  number of kept units
    alive_before [R][B]           int32  |A_r|: tokens alive when round r fires ([R][B][G] when the lists of a
                                         sequence hold different numbers of tokens)
    total_before [R][B]           int32  sequence length when round r fires (block_r ends there)
    Returns (pos [R][B][G][k_max*block] int32 ascending, -1 padded; count [R][B][G]; rc) with
    rc = 0, 1 (inconsistent counts) or 3 (bad kept list); a failing list gets count -1 from
    that round on.
    """
    kept_sorted = np.asarray(kept_sorted, np.int32)
    R, B, G, k_max = kept_sorted.shape
    budget = np.asarray(budget, np.int32).reshape(R, B)
    alive_before = np.asarray(alive_before, np.int32)
    alive_before = alive_before.reshape(R, B, G) if alive_before.size == R * B * G and G > 1 else \
        np.repeat(alive_before.reshape(R, B, 1), G, 2)
    total_before = np.asarray(total_before, np.int32).reshape(R, B)
    pos = np.full((R, B, G, k_max * block), -1, np.int32)
    count = np.full((R, B, G), -1, np.int32)
    rc = 0
    for b in range(B):
        for g in range(G):
            kept_prev = np.zeros(0, np.int64)          # kept_{r-1}, original positions
            for r in range(R):
                n_alive, total, K = int(alive_before[r, b, g]), int(total_before[r, b]), int(budget[r, b])
                grow = n_alive - len(kept_prev)        # |block_r|: tokens appended since the last round
                if grow < 0 or grow > total or K < 0 or K > k_max:
                    rc = max(rc, 1)
                    break
                # A_r = kept_{r-1} U block_r, in cache order; block_r = the last `grow` positions before `total`
                A = np.concatenate([kept_prev, np.arange(total - grow, total, dtype=np.int64)])
                n_units = (n_alive + block - 1) // block
                units = kept_sorted[r, b, g, :K].astype(np.int64)
                if K > n_units or (K and (units.min() < 0 or units.max() >= n_units)) or np.any(np.diff(units) <= 0):
                    rc = max(rc, 3)
                    break
                d = np.zeros(n_alive, bool)            # the paper's decision vector d_r over A_r
                for u in units:
                    d[u * block: min((u + 1) * block, n_alive)] = True
                kept_prev = A[d]
                count[r, b, g] = len(kept_prev)
                pos[r, b, g, : len(kept_prev)] = kept_prev
    return pos, count, rc


def dense_mask(T, total_before, kept_positions):
    """The paper's dense replay mask M [T][T] (bool) of ONE list: `total_before[r]` = sequence length
    when round r fires, `kept_positions[r]` = kept_r in original positions.  Row t marks the keys
    visible when token t was generated."""
    R = len(total_before)
    bounds = [0] + [int(x) for x in total_before] + [T]          # block r spans bounds[r] .. bounds[r+1]
    M = np.zeros((T, T), bool)
    for r in range(R + 1):
        lo, hi = bounds[r], min(bounds[r + 1], T)
        for t in range(lo, hi):
            M[t, lo: t + 1] = True                               # causal inside the block
            if r > 0:
                M[t, np.asarray(kept_positions[r - 1], np.int64)] = True   # every query of block r sees kept_{r-1}
    M[np.arange(T), np.arange(T)] = True                         # the diagonal
    return M


def replay_attention(q, k, v, masks, scale=None):
    """Attention of every token under its replay mask, in float64 (paper Section 4.5: one forward pass
    whose per-layer masks reproduce what each token saw at rollout time).

    q [Hq][T][d], k/v [Hkv][T][d] float64 (ONE layer of ONE sequence), masks [G_l][T][T] bool with
    G_l = 1 (one mask for the layer) or Hkv (one per KV head).  Returns out [Hq][T][d]."""
    Hq, T, d = q.shape
    Hkv = k.shape[0]
    g = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((Hq, T, d))
    for hq in range(Hq):
        h = hq // g
        M = masks[h if masks.shape[0] == Hkv else 0]
        z = (q[hq] @ k[h].T) * scale
        z = np.where(M, z, -np.inf)
        z -= z.max(-1, keepdims=True)
        p = np.exp(z)
        p /= p.sum(-1, keepdims=True)
        out[hq] = p @ v[h]
    return out
