"""Pins for the oracle's cache operations: compaction, ragged decode attention
and the attention-based eviction score.

* compaction: numpy fancy indexing (the definition), the worked example of the
  paper's replay-mask figure (golden file), order preservation, identity;
* decode attention: dense softmax attention over the UNCOMPACTED cache with
  the evicted positions masked (torch's library attention in fp64), textbook
  special cases;
* score: rows of a softmax sum to one, library softmax with an explicit causal
  mask, and a cross-check against the independently written decode routine.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2604_18002_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_cache(dtype, L=2, B=3, Hq=4, Hkv=2, d=16, lens=(9, 1, 14), cap=20, seed=0):
    return synth.make_cache(L, B, Hq, Hkv, d, dtype, list(lens), capacity=cap, seed=seed)


# ------------------------------------------------------------------ compaction

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("lists", [0, 1, 2])
def test_compact_is_fancy_indexing(dtype, lists):
    c = small_cache(dtype)
    k, v = synth.to_numpy(c.k), synth.to_numpy(c.v)
    so, lens = c.seq_off.numpy(), c.lens.numpy()
    G = oracle.lists_G(lists, c.L, c.Hkv)
    rng = np.random.default_rng(lists)
    budget = np.array([5, 1, 7], np.int32)
    ks = -np.ones((c.B, G, 8), np.int32)
    for b in range(c.B):
        for g in range(G):
            ks[b, g, :budget[b]] = np.sort(rng.choice(lens[b], budget[b], replace=False))
    ko, vo, nl, rc = oracle.compact_kv(k, v, so, lens, ks, budget, lists)
    assert rc == 0 and np.array_equal(nl, budget)
    for l in range(c.L):
        for h in range(c.Hkv):
            g = 0 if lists == 0 else (l if lists == 1 else l * c.Hkv + h)
            for b in range(c.B):
                idx = ks[b, g, :budget[b]]
                assert np.array_equal(ko[l, h, so[b]:so[b] + budget[b]], k[l, h, so[b] + idx])
                assert np.array_equal(vo[l, h, so[b]:so[b] + budget[b]], v[l, h, so[b] + idx])


def test_compact_identity_and_order():
    c = small_cache(torch.float32, lens=(6, 6, 6))
    k, v = synth.to_numpy(c.k), synth.to_numpy(c.v)
    ks = np.broadcast_to(np.arange(6, dtype=np.int32), (3, 1, 6)).copy()
    ko, vo, nl, rc = oracle.compact_kv(k, v, c.seq_off.numpy(), c.lens.numpy(), ks, [6, 6, 6], 0)
    so = c.seq_off.numpy()
    for b in range(3):
        assert np.array_equal(ko[:, :, so[b]:so[b] + 6], k[:, :, so[b]:so[b] + 6])
    # rows tagged with their original position stay in ascending order
    k2 = k.copy()
    for t in range(6):
        k2[:, :, so[0] + t, 0] = t
    ks[0, 0] = [1, 2, 4, 5, -1, -1]
    ko, _, nl, _ = oracle.compact_kv(k2, v, so, c.lens.numpy(), ks, [4, 6, 6], 0)
    assert ko[0, 0, so[0]:so[0] + 4, 0].tolist() == [1, 2, 4, 5] and nl[0] == 4


def test_compact_blocks_with_ragged_last_unit():
    c = small_cache(torch.float32, L=1, B=1, Hq=1, Hkv=1, d=4, lens=(11,), cap=16)
    k, v = synth.to_numpy(c.k), synth.to_numpy(c.v)
    ks = np.array([[[0, 2, -1]]], np.int32)          # units of 4 tokens: [0..3], [8..10]
    ko, vo, nl, rc = oracle.compact_kv(k, v, c.seq_off.numpy(), c.lens.numpy(), ks, [2], 0, block=4)
    assert rc == 0 and nl[0] == 7
    assert np.array_equal(ko[0, 0, :7], k[0, 0, [0, 1, 2, 3, 8, 9, 10]])
    # invalid lists are refused
    for bad in ([[2, 0, -1]], [[0, 3, -1]], [[1, 1, -1]]):
        assert oracle.compact_kv(k, v, c.seq_off.numpy(), c.lens.numpy(), np.array([bad], np.int32), [2], 0, block=4)[3] == 3


def test_compact_reproduces_replay_mask_figure():
    """Two eviction rounds of the paper's replay-mask figure, done by compaction:
    the rows that survive must be exactly the keys the figure marks visible."""
    with open(os.path.join(GOLDEN, "replay_mask_figure.json")) as f:
        fig = json.load(f)
    T = fig["tokens"]
    k = np.zeros((1, 1, T, 2), np.float32)
    v = np.zeros((1, 1, T, 2), np.float32)
    so = np.array([0, T], np.int64)
    alive = []           # original token ids currently in the cache, in cache order
    length = 0
    nxt = 0
    for rnd in fig["rounds"]:
        while nxt <= rnd["after_token"]:
            k[0, 0, length, 0] = nxt
            alive.append(nxt)
            length += 1
            nxt += 1
        keep_idx = [i for i, t in enumerate(alive) if t not in rnd["evicts"]]
        ks = np.array([[keep_idx]], np.int32)
        k, v, nl, rc = oracle.compact_kv(k, v, so, np.array([length], np.int32), ks, [len(keep_idx)], 0)
        assert rc == 0
        length = int(nl[0])
        alive = [int(x) for x in k[0, 0, :length, 0]]
        # keys visible to the next generated token = survivors + itself
        row = fig["visible"][str(rnd["after_token"] + 1)]
        assert alive + [rnd["after_token"] + 1] == row
    assert alive == fig["final_survivors"]


# ------------------------------------------------------------------ decode attention

def dense_masked_attention(k, v, q, so, b, keep_mask, scale, Hkv):
    """softmax attention over the whole uncompacted strip with evicted keys masked to -inf
    (torch's fp64 scaled_dot_product_attention, an implementation independent of the oracle)."""
    L, _, _, d = k.shape
    Hq = q.shape[2]
    g = Hq // Hkv
    T = keep_mask.shape[0]
    out = np.zeros((L, Hq, d))
    for l in range(L):
        kk = torch.from_numpy(synth.as_f64(k[l, :, so[b]:so[b] + T]))         # [Hkv][T][d]
        vv = torch.from_numpy(synth.as_f64(v[l, :, so[b]:so[b] + T]))
        qq = torch.from_numpy(synth.as_f64(q[l, b])).reshape(Hq, 1, d)
        kk = kk.repeat_interleave(g, 0)
        vv = vv.repeat_interleave(g, 0)
        m = torch.from_numpy(keep_mask.astype(bool)).reshape(1, 1, T).expand(Hq, 1, T)
        o = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, attn_mask=m, scale=scale)
        out[l] = o.reshape(Hq, d).numpy()
    return out


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_ragged_attention_on_compacted_equals_dense_masked(dtype):
    L, B, Hq, Hkv, d = 2, 3, 6, 2, 32
    lens = [37, 5, 64]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=70, seed=3)
    k, v = synth.to_numpy(c.k), synth.to_numpy(c.v)
    so = c.seq_off.numpy()
    q = synth.to_numpy(synth.make_queries(L, B, Hq, d, dtype, seed=4))
    logits = synth.make_logits(B, 1, 64, seed=5).numpy()
    budget = np.array([20, 2, 21], np.int32)
    ko, ks, km, st = oracle.sample_evict(logits, lens, None, budget, 21, seed=1, rnd=0)
    kc, vc, nl, rc = oracle.compact_kv(k, v, so, c.lens.numpy(), ks, budget, 0)
    assert rc == 0
    scale = 1.0 / math.sqrt(d)
    out, rc = oracle.decode_attn(kc, vc, so, nl.copy(), q, scale=scale)
    assert rc == 0
    for b in range(B):
        ref = dense_masked_attention(k, v, q, so, b, km[b, 0, :lens[b]], scale, Hkv)
        assert np.allclose(out[:, b], ref, rtol=1e-10, atol=1e-12)


def test_attention_special_cases():
    L, B, Hq, Hkv, d = 1, 1, 2, 1, 8
    rng = np.random.default_rng(0)
    so = np.array([0, 16], np.int64)
    k = rng.normal(size=(L, Hkv, 16, d)).astype(np.float32)
    v = rng.normal(size=(L, Hkv, 16, d)).astype(np.float32)
    q = rng.normal(size=(L, B, Hq, d)).astype(np.float32)
    # one row: output is that value row
    out, _ = oracle.decode_attn(k.copy(), v.copy(), so, np.array([1], np.int32), q)
    assert np.allclose(out[0, 0], np.stack([v[0, 0, 0]] * 2), atol=1e-15)
    # equal keys: output is the mean of the values
    k2 = np.broadcast_to(k[:, :, :1], k.shape).copy()
    out, _ = oracle.decode_attn(k2, v.copy(), so, np.array([10], np.int32), q)
    assert np.allclose(out[0, 0, 0], v[0, 0, :10].astype(np.float64).mean(0), atol=1e-14)
    # one dominant key
    k3 = k.copy()
    k3[0, 0, 4] = 200.0 * q[0, 0, 0] / np.linalg.norm(q[0, 0, 0])
    out, _ = oracle.decode_attn(k3, v.copy(), so, np.array([12], np.int32), q)
    assert np.allclose(out[0, 0, 0], v[0, 0, 4], atol=1e-9)
    # permuting cache rows leaves the output unchanged
    perm = rng.permutation(12)
    k4, v4 = k.copy(), v.copy()
    k4[0, 0, :12] = k[0, 0, perm]
    v4[0, 0, :12] = v[0, 0, perm]
    a, _ = oracle.decode_attn(k.copy(), v.copy(), so, np.array([12], np.int32), q)
    b_, _ = oracle.decode_attn(k4, v4, so, np.array([12], np.int32), q)
    assert np.allclose(a, b_, atol=1e-14)
    # empty cache: zeros
    out, _ = oracle.decode_attn(k.copy(), v.copy(), so, np.array([0], np.int32), q)
    assert not out.any()


def test_attention_append_semantics():
    L, B, Hq, Hkv, d = 2, 2, 4, 2, 8
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.float32, [5, 3], capacity=8, seed=1)
    k, v = synth.to_numpy(c.k).copy(), synth.to_numpy(c.v).copy()
    so = c.seq_off.numpy()
    q = synth.to_numpy(synth.make_queries(L, B, Hq, d, torch.float32, seed=2))
    nk, nv = synth.make_new_kv(L, B, Hkv, d, torch.float32, seed=3)
    nk, nv = nk.numpy(), nv.numpy()
    lens = np.array([5, 3], np.int32)
    k_app, v_app = k.copy(), v.copy()
    out, rc = oracle.decode_attn(k_app, v_app, so, lens, q, nk, nv)
    assert rc == 0 and lens.tolist() == [6, 4]
    # the same thing by hand: write the rows, then attend over len+1 rows
    k_ref, v_ref = k.copy(), v.copy()
    for b, T in enumerate([5, 3]):
        k_ref[:, :, so[b] + T] = nk[:, b]
        v_ref[:, :, so[b] + T] = nv[:, b]
    assert np.array_equal(k_app, k_ref) and np.array_equal(v_app, v_ref)
    ref, _ = oracle.decode_attn(k_ref, v_ref, so, np.array([6, 4], np.int32), q)
    assert np.array_equal(out, ref)
    # layer ranges: lens moves only with the call that covers the last layer
    lens = np.array([5, 3], np.int32)
    k2, v2 = k.copy(), v.copy()
    o1, _ = oracle.decode_attn(k2, v2, so, lens, q, nk, nv, layer_begin=0, layer_end=1)
    assert lens.tolist() == [5, 3]
    o2, _ = oracle.decode_attn(k2, v2, so, lens, q, nk, nv, layer_begin=1, layer_end=2)
    assert lens.tolist() == [6, 4]
    assert np.array_equal(o1[0], out[0]) and np.array_equal(o2[1], out[1])
    # no room left
    lens = np.array([8, 3], np.int32)
    assert oracle.decode_attn(k.copy(), v.copy(), so, lens, q, nk, nv)[1] == 4


# ------------------------------------------------------------------ score

def library_score(k, q_recent, so, b, T, lists, Hkv, block):
    """psi via torch.softmax (fp64) with an explicit causal mask; block mean via numpy."""
    L = k.shape[0]
    Hq, w, d = q_recent.shape[2:]
    g = Hq // Hkv
    G = oracle.lists_G(lists, L, Hkv)
    psi = np.zeros((G, T))
    rows = np.zeros(G)
    for l in range(L):
        for hq in range(Hq):
            h = hq // g
            gi = 0 if lists == 0 else (l if lists == 1 else l * Hkv + h)
            K = torch.from_numpy(synth.as_f64(k[l, h, so[b]:so[b] + T]))
            Q = torch.from_numpy(synth.as_f64(q_recent[l, b, hq]))
            z = (Q @ K.T) / math.sqrt(d)
            pos = torch.arange(T - w, T).reshape(w, 1)
            z = z.masked_fill(torch.arange(T).reshape(1, T) > pos, float("-inf"))
            valid = (pos >= 0).reshape(w)
            A = torch.softmax(z[valid], -1)
            psi[gi] += A.sum(0).numpy()
            rows[gi] += int(valid.sum())
    psi /= rows[:, None]
    n = (T + block - 1) // block
    return np.stack([[psi[gi, u * block:min((u + 1) * block, T)].mean() for u in range(n)] for gi in range(G)])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("lists,block", [(0, 1), (1, 4), (2, 1), (2, 5)])
def test_score_matches_library_softmax(dtype, lists, block):
    L, B, Hq, Hkv, d, w = 2, 3, 4, 2, 16, 5
    lens = [23, 3, 40]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=40, seed=6)
    k = synth.to_numpy(c.k)
    so = c.seq_off.numpy()
    qr = synth.to_numpy(synth.normal((L, B, Hq, w, d), 7, dtype))
    s = oracle.score_evict(k, so, c.lens.numpy(), qr, block, lists)
    for b in range(B):
        ref = library_score(k, qr, so, b, lens[b], lists, Hkv, block)
        n = ref.shape[1]
        assert np.allclose(s[b, :, :n], ref, rtol=1e-11, atol=1e-14)
        assert np.all(np.isnan(s[b, :, n:]))
        # psi is a mean of probability rows: block means weighted by block size sum to 1
        sizes = np.array([min((u + 1) * block, lens[b]) - u * block for u in range(n)])
        assert np.allclose((s[b, :, :n] * sizes).sum(-1), 1.0, atol=1e-12)
    s_log = oracle.score_evict(k, so, c.lens.numpy(), qr, block, lists, log_transform=1)
    m = ~np.isnan(s)
    assert np.allclose(s_log[m], np.log(s[m]), atol=1e-12)


def test_score_equal_keys_gives_causal_uniform():
    L, B, Hq, Hkv, d, w, T = 1, 1, 2, 1, 8, 3, 10
    k = np.ones((L, Hkv, T, d), np.float32)
    qr = np.random.default_rng(0).normal(size=(L, B, Hq, w, d)).astype(np.float32)
    s = oracle.score_evict(k, np.array([0, T], np.int64), np.array([T], np.int32), qr, 1, 0)[0, 0]
    # query j sits at position T-w+j and spreads 1/(pos+1) over keys 0..pos
    want = np.zeros(T)
    for j in range(w):
        pos = T - w + j
        want[:pos + 1] += 1.0 / (pos + 1) / w
    assert np.allclose(s, want, atol=1e-14)


def test_score_single_query_equals_decode_attention_weights():
    """w = 1 and one KV-head group: psi is the decode-attention weight vector.  The decode
    routine reveals its weights when V is the identity (out = p)."""
    L, B, Hq, Hkv, T = 1, 1, 3, 1, 12
    d = 16
    rng = np.random.default_rng(3)
    k = rng.normal(size=(L, Hkv, T, d)).astype(np.float32)
    v = np.zeros((L, Hkv, T, d), np.float32)
    v[0, 0, np.arange(T), np.arange(T)] = 1.0
    q = rng.normal(size=(L, B, Hq, d)).astype(np.float32)
    so = np.array([0, T], np.int64)
    out, _ = oracle.decode_attn(k.copy(), v, so, np.array([T], np.int32), q, scale=1 / math.sqrt(d))
    weights = out[0, 0, :, :T].mean(0)                      # mean over the heads of the group
    s = oracle.score_evict(k, so, np.array([T], np.int32), q.reshape(L, B, Hq, 1, d), 1, 2)[0, 0]
    assert np.allclose(s, weights, atol=1e-14)


# ------------------------------------------------------------------ gradient of the eviction scores

def _score_loss(k, so, lens, qr, block, lists, up, log_transform):
    s = oracle.score_evict(k, so, lens, qr, block, lists, log_transform=log_transform, n_max=up.shape[2])
    return float(np.nansum(np.where(np.isnan(s), 0.0, s) * up))


@pytest.mark.parametrize("lists,block,log_transform", [(0, 1, 0), (1, 3, 0), (2, 1, 1), (1, 4, 1)])
def test_score_grad_matches_finite_differences(lists, block, log_transform):
    """Central differences of the (separately pinned) forward scores, on fp32 inputs."""
    rng = np.random.default_rng(7 + lists)
    L, B, Hq, Hkv, d, w = 2, 2, 4, 2, 8, 3
    lens = np.array([7, 2], np.int32)                       # the second sequence is shorter than the window
    so = np.array([0, 8, 11], np.int64)
    k = rng.normal(0, 1, (L, Hkv, 11, d)).astype(np.float32)
    qr = rng.normal(0, 1, (L, B, Hq, w, d)).astype(np.float32)
    G = oracle.lists_G(lists, L, Hkv)
    n_max = (8 + block - 1) // block
    up = rng.normal(0, 1, (B, G, n_max))
    gq, gk = oracle.score_evict_grad(k, so, lens, qr, block, lists, up, log_transform=log_transform)
    h = 2.0 ** -9
    for _ in range(40):
        if rng.random() < 0.5:
            idx = tuple(rng.integers(0, s) for s in qr.shape)
            a, b2 = qr.copy(), qr.copy()
            a[idx] += h
            b2[idx] -= h
            fd = (_score_loss(k, so, lens, a, block, lists, up, log_transform) - _score_loss(k, so, lens, b2, block, lists, up, log_transform)) / \
                 (float(a[idx]) - float(b2[idx]))
            assert abs(fd - gq[idx]) <= 1e-4 * max(1.0, abs(fd)), ("q", idx)
        else:
            idx = tuple(rng.integers(0, s) for s in k.shape)
            a, b2 = k.copy(), k.copy()
            a[idx] += h
            b2[idx] -= h
            fd = (_score_loss(a, so, lens, qr, block, lists, up, log_transform) - _score_loss(b2, so, lens, qr, block, lists, up, log_transform)) / \
                 (float(a[idx]) - float(b2[idx]))
            assert abs(fd - gk[idx]) <= 1e-4 * max(1.0, abs(fd)), ("k", idx)
    # rows beyond a sequence's length and queries before its start get no gradient
    assert np.all(gk[:, :, 7:8] == 0) and np.all(gk[:, :, 10:] == 0) and np.all(gq[:, 1, :, 0] == 0)


def test_score_grad_vanishes_along_the_normalisation():
    """sum_j |B_j| s_j = 1 whatever q and k are: an upstream gradient proportional to the unit sizes gives zero."""
    rng = np.random.default_rng(2)
    L, B, Hq, Hkv, d, w, block = 1, 1, 4, 2, 16, 5, 4
    lens = np.array([14], np.int32)
    so = np.array([0, 14], np.int64)
    k = rng.normal(0, 1, (L, Hkv, 14, d)).astype(np.float32)
    qr = rng.normal(0, 1, (L, B, Hq, w, d)).astype(np.float32)
    up = np.array([[[4, 4, 4, 2]]], np.float64) * 0.37             # unit sizes 4, 4, 4, 2
    gq, gk = oracle.score_evict_grad(k, so, lens, qr, block, 1, up)
    assert np.max(np.abs(gq)) <= 1e-12 and np.max(np.abs(gk)) <= 1e-12
    up2 = up.copy()
    up2[0, 0, 1] += 1.0
    gq2, gk2 = oracle.score_evict_grad(k, so, lens, qr, block, 1, up2)
    assert np.max(np.abs(gq2)) > 1e-4 and np.max(np.abs(gk2)) > 1e-4
