"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the
same seeded inputs.  Integer outputs bit-exact; eviction log-probs <= 1e-3 abs;
attention <= 1e-5 abs (fp32) / <= 2e-2 relative per output vector (bf16 K/V,
fp32 accumulate); scores <= 1e-5 abs (fp32) / 2e-2 of the largest score (bf16)."""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import gpu_logprob, gpu_logprob_grad, gpu_sample, max_rel_err_per_vector, ngc, status_value, to_device_cache
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu

TOL_ATTN_F32 = 1e-5
TOL_ATTN_BF16 = 2e-2
TOL_LOGP = 1e-3


# ------------------------------------------------------------------ sample

@pytest.mark.parametrize("B,G,n_max,std", [(3, 2, 100, 1.0), (4, 1, 512, 1.0), (2, 3, 4096, 1.4142), (2, 2, 16384, 1.0),
                                            (5, 1, 1, 1.0), (3, 1, 33, 0.0)])
def test_sample_bit_exact(B, G, n_max, std):
    rng = np.random.default_rng(n_max)
    logits = synth.make_logits(B, G, n_max, seed=n_max, std=max(std, 1e-9)).numpy()
    if std == 0.0:
        logits[:] = 0.25                      # all ties in greedy mode below
    n = rng.integers(max(1, n_max // 2), n_max + 1, B).astype(np.int32)
    n[0] = n_max
    P = np.array([rng.integers(0, x // 4 + 1) for x in n], np.int32)
    K = np.array([rng.integers(p, x + 1) for p, x in zip(P, n)], np.int32)
    K[0] = max(P[0], n[0] // 2)
    k_max = int(K.max()) + 3
    for greedy in (0, 1):
        ref = oracle.sample_evict(logits, n, P, K, k_max, seed=77, rnd=5, greedy=greedy, list_base=11)
        got = gpu_sample(logits, n, P, K, k_max, seed=77, rnd=5, greedy=greedy, list_base=11)
        assert got[3] == 0 and not ref[3].any()
        assert np.array_equal(got[0], ref[0]), "kept_order"
        assert np.array_equal(got[1], ref[1]), "kept_sorted"
        assert np.array_equal(got[2], ref[2]), "keep_mask"


@pytest.mark.parametrize("kind", ["quantised", "constant", "infinite", "few_distinct"])
def test_sample_long_lists_with_ties_around_the_selection_threshold(kind):
    """Lists long enough for the pre-selection of drawable candidates (more than 8192 candidates, at most three
    quarters drawn): equal keys at the threshold must still go to the smaller index, and budgets on both sides of
    the three-quarter rule take both code paths."""
    B, G, n_max = 6, 2, 16384
    rng = np.random.default_rng(5)
    logits = synth.make_logits(B, G, n_max, seed=21).numpy()
    if kind == "quantised":
        logits = np.round(logits * 4.0).astype(np.float32) / 4.0          # many exact ties (greedy), few in sampled mode
    elif kind == "constant":
        logits[:] = -1.5
    elif kind == "infinite":
        logits[:, :, ::3] = -np.inf
        logits[:, :, 5::97] = np.inf
    else:
        logits = rng.integers(0, 3, logits.shape).astype(np.float32)      # three distinct values
    n = np.array([16384, 16384, 12000, 8193, 9000, 16000], np.int32)
    P = np.array([0, 100, 0, 1, 0, 4000], np.int32)
    K = np.array([8192, 8292, 9000, 4097, 6751, 13000], np.int32)          # list 4: just over three quarters; list 5: P > 0
    k_max = int(K.max())
    for greedy in (1, 0):
        ref = oracle.sample_evict(logits, n, P, K, k_max, seed=9, rnd=3, greedy=greedy, list_base=2)
        got = gpu_sample(logits, n, P, K, k_max, seed=9, rnd=3, greedy=greedy, list_base=2)
        assert got[3] == 0 and not ref[3].any()
        for i in range(3):
            assert np.array_equal(got[i], ref[i]), (kind, greedy, i)


def test_sample_large_list_uses_workspace():
    B, G, n_max = 2, 1, 40000
    logits = synth.make_logits(B, G, n_max, seed=3).numpy()
    n = np.array([40000, 17000], np.int32)
    K = np.array([13000, 17000], np.int32)
    ref = oracle.sample_evict(logits, n, None, K, 17000, seed=1, rnd=2)
    got = gpu_sample(logits, n, None, K, 17000, seed=1, rnd=2)
    assert got[3] == 0
    for i in range(3):
        assert np.array_equal(got[i], ref[i])


def test_sample_edge_cases_and_status():
    logits = synth.make_logits(4, 1, 64, seed=9).numpy()
    # K = n (keep all), K = P (draw nothing), n = 0, K = 0
    n = np.array([64, 40, 0, 10], np.int32)
    P = np.array([0, 7, 0, 0], np.int32)
    K = np.array([64, 7, 0, 0], np.int32)
    ref = oracle.sample_evict(logits, n, P, K, 64, seed=4, rnd=4)
    got = gpu_sample(logits, n, P, K, 64, seed=4, rnd=4)
    assert got[3] == 0
    for i in range(3):
        assert np.array_equal(got[i], ref[i])
    # infinities order first / last
    logits[0, 0, 5] = np.inf
    logits[0, 0, 9] = -np.inf
    ref = oracle.sample_evict(logits, n, P, K, 64, seed=4, rnd=4)
    got = gpu_sample(logits, n, P, K, 64, seed=4, rnd=4)
    assert np.array_equal(got[0], ref[0]) and got[0][0, 0, 0] == 5 and got[0][0, 0, 63] == 9
    # NaN candidate -> status 2, list blanked, other lists unaffected
    logits[1, 0, 20] = np.nan
    ref = oracle.sample_evict(logits, n, P, K, 64, seed=4, rnd=4)
    got = gpu_sample(logits, n, P, K, 64, seed=4, rnd=4)
    assert got[3] == 2 and ref[3][1, 0] == 2
    for i in range(3):
        assert np.array_equal(got[i], ref[i])
    # bad counts -> status 1
    logits[1, 0, 20] = 0
    got = gpu_sample(logits, n, P, np.array([65, 7, 0, 0], np.int32), 64, seed=4, rnd=4)
    assert got[3] == 1 and np.all(got[0][0] == -1) and np.all(got[1][0] == -1) and got[2][0].sum() == 0
    assert np.array_equal(got[0][1:], ref[0][1:])


# ------------------------------------------------------------------ log-prob

@pytest.mark.parametrize("NB,B,G,n_max,frac", [(1, 3, 2, 700, 0.5), (4, 2, 3, 768, 1 / 3), (1, 2, 1, 4096, 0.5),
                                                (1, 1, 2, 16384, 0.5), (2, 2, 1, 40, 1.0)])
def test_logprob_matches_oracle(NB, B, G, n_max, frac):
    rng = np.random.default_rng(n_max + NB)
    logits = synth.make_logits(NB * B, G, n_max, seed=n_max, std=1.5).numpy().reshape(NB, B, G, n_max)
    n = rng.integers(n_max // 2, n_max + 1, (NB, B)).astype(np.int32)
    P = rng.integers(0, 5, (NB, B)).astype(np.int32)
    K = np.maximum(P, np.ceil(n * frac).astype(np.int32))
    k_max = int(K.max())
    ko = np.stack([oracle.sample_evict(logits[r], n[r], P[r], K[r], k_max, seed=3, rnd=r)[0] for r in range(NB)])
    ref, rc = oracle.evict_logprob(logits, n, P, K, ko)
    assert rc == 0
    got, st = gpu_logprob(logits, n, P, K, ko)
    assert st == 0
    assert np.max(np.abs(got - ref)) <= TOL_LOGP
    assert np.max(np.abs(got - ref)) <= 1e-7 * np.max(np.abs(ref)) + 1e-9      # fp64 path: far inside the bar


def test_logprob_mask_order_variant_and_bad_lists():
    n_max = 300
    logits = synth.make_logits(2, 1, n_max, seed=1).numpy()
    n = np.array([300, 200], np.int32)
    K = np.array([100, 50], np.int32)
    ko, ks, km, _ = oracle.sample_evict(logits, n, None, K, 100, seed=8, rnd=0)
    # a caller that only stored the mask passes ascending order: same kernel
    ref, _ = oracle.evict_logprob(logits, n, None, K, ks)
    got, st = gpu_logprob(logits, n, None, K, ks)
    assert st == 0 and np.max(np.abs(got - ref)) <= 1e-8
    bad = ko.copy()
    bad[1, 0, 3] = bad[1, 0, 4]                   # repeated unit
    got, st = gpu_logprob(logits, n, None, K, bad)
    assert st == 3 and math.isnan(got[0, 1, 0]) and abs(got[0, 0, 0] - oracle.evict_logprob(logits, n, None, K, ko)[0][0, 0, 0]) < 1e-8
    got, st = gpu_logprob(logits, n, None, np.array([100, 201], np.int32), ko)
    assert st == 1 and math.isnan(got[0, 1, 0])


# ------------------------------------------------------------------ compaction

def run_compact(c, ks, budget, lists, block=1):
    b = ngc()
    dc = to_device_cache(c)
    st = b.new_status()
    b.ngc_compact_kv(dc, torch.as_tensor(ks).cuda(), torch.as_tensor(np.asarray(budget, np.int32)).cuda(), lists, block, status=st)
    torch.cuda.synchronize()
    return dc, status_value(st)


def assert_cache_rows_equal(dc, k_ref, v_ref, so, new_lens):
    k = synth.to_numpy(dc.k)
    v = synth.to_numpy(dc.v)
    for b in range(len(new_lens)):
        sl = slice(int(so[b]), int(so[b]) + int(new_lens[b]))
        assert np.array_equal(k[:, :, sl], k_ref[:, :, sl]), f"K rows of sequence {b}"
        assert np.array_equal(v[:, :, sl], v_ref[:, :, sl]), f"V rows of sequence {b}"


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 64), (torch.bfloat16, 64), (torch.float32, 128)])
@pytest.mark.parametrize("lists", [0, 1, 2])
def test_compact_bit_exact(dtype, d, lists):
    L, B, Hq, Hkv = 3, 4, 4, 2
    lens = [700, 1, 333, 64]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=[800, 4, 333, 100], seed=5)
    G = oracle.lists_G(lists, L, Hkv)
    logits = synth.make_logits(B, G, 700, seed=6).numpy()
    budget = np.array([350, 1, 111, 64], np.int32)       # half, keep-all (len 1), a third, identity
    ko, ks, km, st = oracle.sample_evict(logits, lens, None, budget, 350, seed=2, rnd=0)
    k_ref, v_ref, nl, rc = oracle.compact_kv(synth.to_numpy(c.k), synth.to_numpy(c.v), c.seq_off.numpy(), c.lens.numpy(),
                                             ks, budget, lists)
    assert rc == 0
    dc, st = run_compact(c, ks, budget, lists)
    assert st == 0
    assert np.array_equal(dc.lens.cpu().numpy(), nl)
    assert_cache_rows_equal(dc, k_ref, v_ref, c.seq_off.numpy(), nl)


def test_compact_blocks_ragged_and_corrupt_lists():
    L, B, Hq, Hkv, d = 2, 3, 2, 1, 128
    lens = [1000, 37, 512]
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.bfloat16, lens, capacity=1024, seed=7)
    block = 32
    n_units = [(x + block - 1) // block for x in lens]
    budget = np.array([16, 2, 8], np.int32)
    logits = synth.make_logits(B, 1, 32, seed=8).numpy()
    # keep the ragged last unit of sequences 0 and 1 for sure
    logits[0, 0, n_units[0] - 1] = 50
    logits[1, 0, n_units[1] - 1] = 50
    ko, ks, km, st = oracle.sample_evict(logits, n_units, None, budget, 16, seed=1, rnd=1, greedy=1)
    k_ref, v_ref, nl, rc = oracle.compact_kv(synth.to_numpy(c.k), synth.to_numpy(c.v), c.seq_off.numpy(), c.lens.numpy(),
                                             ks, budget, 0, block=block)
    assert rc == 0 and nl[0] == 15 * 32 + (1000 - 31 * 32) and nl[1] == 37
    dc, st = run_compact(c, ks, budget, 0, block)
    assert st == 0 and np.array_equal(dc.lens.cpu().numpy(), nl)
    assert_cache_rows_equal(dc, k_ref, v_ref, c.seq_off.numpy(), nl)
    # a corrupt list: reported, that sequence untouched (lens too), the others compacted
    bad = ks.copy()
    bad[2, 0, 3] = bad[2, 0, 2]
    dc, st = run_compact(c, bad, budget, 0, block)
    assert st == 3
    lens_after = dc.lens.cpu().numpy()
    assert lens_after[2] == 512 and lens_after[0] == nl[0]
    so = c.seq_off.numpy()
    assert np.array_equal(synth.to_numpy(dc.k)[:, :, so[2]:so[2] + 512], synth.to_numpy(c.k)[:, :, so[2]:so[2] + 512])


def test_compact_per_list_disagreement_is_reported():
    L, B, Hq, Hkv, d = 2, 1, 1, 1, 64
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.float32, [10], capacity=12, seed=1)
    ks = np.array([[[0, 2], [1, 2]]], np.int32)            # units of 4: layer 0 keeps the short last unit + unit 0, ...
    ks[0, 1] = [0, 1]                                      # ... layer 1 keeps two full units: 6 vs 8 tokens
    dc, st = run_compact(c, ks, [2], 1, block=4)
    assert st == 5 and int(dc.lens.item()) == 10
    # the sequence is left exactly as it was: no strip of it moved
    assert torch.equal(dc.k.cpu(), c.k) and torch.equal(dc.v.cpu(), c.v)


def test_compact_sequence_with_one_corrupt_list_is_left_whole():
    """Several lists per sequence, one length per sequence: if one of a sequence's lists is corrupt, none of its strips
    may move (a half-compacted sequence whose length still says the old value would be unusable); the other sequences
    are compacted as usual."""
    L, B, Hq, Hkv, d = 3, 2, 2, 1, 128
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.bfloat16, [64, 48], capacity=64, seed=12)
    logits = synth.make_logits(B, L, 64, seed=13).numpy()
    budget = np.array([20, 16], np.int32)
    ko, ks, km, st = oracle.sample_evict(logits, [64, 48], None, budget, 20, seed=4, rnd=0)
    bad = ks.copy()
    bad[0, 1, 5] = 64                                      # layer 1 of sequence 0: a unit beyond the cache
    dc, st = run_compact(c, bad, budget, 1)
    assert st == 3
    so = c.seq_off.numpy()
    assert list(dc.lens.cpu().numpy()) == [64, 16]
    assert torch.equal(dc.k.cpu()[:, :, :so[1]], c.k[:, :, :so[1]]) and torch.equal(dc.v.cpu()[:, :, :so[1]], c.v[:, :, :so[1]])
    k_ref, v_ref, nl, rc = oracle.compact_kv(synth.to_numpy(c.k), synth.to_numpy(c.v), so, c.lens.numpy(), ks, budget, 1)
    assert rc == 0
    sl = slice(so[1], so[1] + 16)
    assert np.array_equal(synth.to_numpy(dc.k)[:, :, sl], k_ref[:, :, sl]) and np.array_equal(synth.to_numpy(dc.v)[:, :, sl], v_ref[:, :, sl])


# ------------------------------------------------------------------ decode attention

def run_decode(c, q, new_k=None, new_v=None, layer_ranges=None, out_dtype=torch.float32, max_len=None):
    b = ngc()
    dc = to_device_cache(c, max_len)
    qd = q.cuda()
    out = torch.full(q.shape, float("nan"), dtype=out_dtype, device="cuda")
    st = b.new_status()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, dc))
    nk = None if new_k is None else new_k.cuda()
    nv = None if new_v is None else new_v.cuda()
    for (lb, le) in (layer_ranges or [(0, c.L)]):
        b.ngc_decode_attn_ragged(dc, qd, out, nk, nv, lb, le, ws=ws, status=st)
    torch.cuda.synchronize()
    return dc, out.float().cpu().numpy(), status_value(st)


def oracle_decode(c, q, new_k=None, new_v=None):
    k, v = synth.to_numpy(c.k).copy(), synth.to_numpy(c.v).copy()
    lens = c.lens.numpy().copy()
    out, rc = oracle.decode_attn(k, v, c.seq_off.numpy(), lens, synth.to_numpy(q),
                                 None if new_k is None else synth.to_numpy(new_k),
                                 None if new_v is None else synth.to_numpy(new_v))
    return k, v, lens, out, rc


@pytest.mark.parametrize("dtype,d,Hq,Hkv,tol", [
    (torch.float32, 64, 4, 4, TOL_ATTN_F32), (torch.float32, 128, 6, 2, TOL_ATTN_F32),
    (torch.bfloat16, 128, 12, 2, TOL_ATTN_BF16), (torch.bfloat16, 128, 28, 4, TOL_ATTN_BF16),
    (torch.bfloat16, 128, 16, 1, TOL_ATTN_BF16), (torch.bfloat16, 128, 2, 2, TOL_ATTN_BF16),
    (torch.bfloat16, 64, 8, 2, TOL_ATTN_BF16), (torch.bfloat16, 128, 40, 2, TOL_ATTN_BF16)])
def test_decode_matches_oracle(dtype, d, Hq, Hkv, tol):
    L, B = 2, 5
    lens = [1, 63, 64, 65, 700]                  # one row, tile edges, several tiles with a ragged tail
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=[2, 64, 66, 128, 800], seed=11,
                         outlier_channels=4 if d == 128 else 0)
    q = synth.make_queries(L, B, Hq, d, dtype, seed=12)
    _, _, _, ref, rc = oracle_decode(c, q)
    assert rc == 0
    dc, got, st = run_decode(c, q)
    assert st == 0
    if dtype == torch.float32:
        assert np.max(np.abs(got - ref)) <= tol
    else:
        assert max_rel_err_per_vector(got, ref) <= tol
    assert np.array_equal(dc.lens.cpu().numpy(), np.array(lens, np.int32))


@pytest.mark.parametrize("dtype,d,Hq,Hkv", [(torch.float32, 64, 4, 4), (torch.bfloat16, 128, 12, 2)])
def test_decode_append_and_layer_ranges(dtype, d, Hq, Hkv):
    L, B = 4, 3
    lens = [0, 127, 300]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=[1, 128, 310], seed=13)
    q = synth.make_queries(L, B, Hq, d, dtype, seed=14)
    nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=15)
    k_ref, v_ref, lens_ref, ref, rc = oracle_decode(c, q, nk, nv)
    assert rc == 0 and lens_ref.tolist() == [1, 128, 301]
    for ranges in ([(0, L)], [(0, 1), (1, 3), (3, L)]):
        dc, got, st = run_decode(c, q, nk, nv, layer_ranges=ranges)
        assert st == 0
        assert np.array_equal(dc.lens.cpu().numpy(), lens_ref)
        kg, vg = synth.to_numpy(dc.k), synth.to_numpy(dc.v)
        so = c.seq_off.numpy()
        for b in range(B):
            sl = slice(int(so[b]), int(so[b]) + int(lens_ref[b]))
            assert np.array_equal(kg[:, :, sl], k_ref[:, :, sl]) and np.array_equal(vg[:, :, sl], v_ref[:, :, sl])
        if dtype == torch.float32:
            assert np.max(np.abs(got - ref)) <= TOL_ATTN_F32
        else:
            assert max_rel_err_per_vector(got, ref) <= TOL_ATTN_BF16


def test_decode_full_strip_is_reported_and_skipped():
    L, B, Hq, Hkv, d = 1, 2, 2, 1, 64
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.float32, [8, 5], capacity=8, seed=1)
    q = synth.make_queries(L, B, Hq, d, torch.float32, seed=2)
    nk, nv = synth.make_new_kv(L, B, Hkv, d, torch.float32, seed=3)
    dc, got, st = run_decode(c, q, nk, nv)
    assert st == 4
    assert dc.lens.cpu().tolist() == [8, 6]
    assert not got[0, 0].any()                       # the full sequence is skipped
    # the other sequence is served as usual: compare with the oracle on a cache where sequence 0 has room
    c2 = c.clone()
    c2.lens[0] = 7
    _, _, _, ref, rc = oracle_decode(c2, q, nk, nv)
    assert rc == 0 and np.max(np.abs(got[0, 1] - ref[0, 1])) <= TOL_ATTN_F32


def test_decode_dead_rows_with_nan_do_not_leak():
    """Rows beyond lens hold unspecified bytes: fill them with NaN/Inf patterns."""
    L, B, Hq, Hkv, d = 1, 2, 12, 2, 128
    lens = [70, 200]
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.bfloat16, lens, capacity=256, seed=21)
    so = c.seq_off.numpy()
    for b in range(B):
        c.k[:, :, so[b] + lens[b]:so[b + 1]] = float("nan")
        c.v[:, :, so[b] + lens[b]:so[b + 1]] = float("inf")
    q = synth.make_queries(L, B, Hq, d, torch.bfloat16, seed=22)
    _, _, _, ref, _ = oracle_decode(c, q)
    _, got, st = run_decode(c, q)
    assert st == 0 and np.isfinite(got).all()
    assert max_rel_err_per_vector(got, ref) <= TOL_ATTN_BF16


def test_decode_bf16_output_and_token_splits():
    # few strips and long sequences: the launch splits along tokens and combines
    L, B, Hq, Hkv, d = 1, 2, 12, 2, 128
    lens = [5000, 1300]
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.bfloat16, lens, capacity=5001, seed=31, outlier_channels=4)
    q = synth.make_queries(L, B, Hq, d, torch.bfloat16, seed=32)
    _, _, _, ref, _ = oracle_decode(c, q)
    b = ngc()
    assert b.workspace_bytes(b.OP_DECODE, to_device_cache(c)) > 0
    _, got, st = run_decode(c, q)
    assert st == 0 and max_rel_err_per_vector(got, ref) <= TOL_ATTN_BF16
    _, got16, st = run_decode(c, q, out_dtype=torch.bfloat16)
    assert st == 0 and max_rel_err_per_vector(got16, ref) <= TOL_ATTN_BF16 + 2 ** -8
    # fp32 cache with splits
    c32 = synth.make_cache(1, 2, 4, 4, 64, torch.float32, [3000, 900], capacity=3000, seed=33)
    q32 = synth.make_queries(1, 2, 4, 64, torch.float32, seed=34)
    _, _, _, ref32, _ = oracle_decode(c32, q32)
    _, got32, st = run_decode(c32, q32)
    assert st == 0 and np.max(np.abs(got32 - ref32)) <= TOL_ATTN_F32


# ------------------------------------------------------------------ score

@pytest.mark.parametrize("dtype,d,Hq,Hkv", [(torch.float32, 64, 4, 4), (torch.bfloat16, 128, 12, 2), (torch.bfloat16, 128, 28, 4)])
@pytest.mark.parametrize("lists,block", [(0, 1), (1, 32), (2, 1), (1, 5)])
def test_score_matches_oracle(dtype, d, Hq, Hkv, lists, block):
    L, B, w = 2, 4, 5
    lens = [3, 256, 257, 900]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=1000, seed=41)
    qr = synth.normal((L, B, Hq, w, d), 42, dtype)
    n_max = (900 + block - 1) // block
    ref = oracle.score_evict(synth.to_numpy(c.k), c.seq_off.numpy(), c.lens.numpy(), synth.to_numpy(qr), block, lists, n_max=n_max)
    b = ngc()
    dc = to_device_cache(c)
    G = oracle.lists_G(lists, L, Hkv)
    logits = torch.full((B, G, n_max), -5.0, dtype=torch.float32, device="cuda")
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE, dc, G, n_max))
    st = b.new_status()
    b.ngc_score_evict(dc, qr.cuda(), block, lists, logits, ws=ws, status=st)
    torch.cuda.synchronize()
    got = logits.cpu().numpy().astype(np.float64)
    live = ~np.isnan(ref)
    assert np.all(got[~live] == -5.0)                 # units beyond the sequence are untouched
    if dtype == torch.float32:
        assert np.max(np.abs(got[live] - ref[live])) <= 1e-5
    else:
        for bb in range(B):
            for g in range(G):
                m = live[bb, g]
                assert np.max(np.abs(got[bb, g][m] - ref[bb, g][m])) <= 2e-2 * ref[bb, g][m].max()
    # log transform
    b.ngc_score_evict(dc, qr.cuda(), block, lists, logits, log_transform=1, ws=ws, status=st)
    torch.cuda.synchronize()
    got_log = logits.cpu().numpy().astype(np.float64)
    assert np.allclose(got_log[live], np.log(got[live]), atol=1e-5)


@pytest.mark.parametrize("Hq,Hkv,w,lens", [(12, 2, 1, [1, 63, 64, 2000]), (12, 2, 3, [2, 65, 128, 1500]), (28, 4, 5, [4, 5, 6, 3000]),
                                            (8, 1, 5, [700, 64, 1, 129]), (16, 2, 7, [900, 10, 3, 300]), (4, 4, 6, [5, 6, 7, 2100])])
def test_score_window_sizes_and_ragged_lengths(Hq, Hkv, w, lens):
    """bf16, d = 128: the tensor-core path (rows per strip <= 40) and the plain path (more rows), windows
    shorter and longer than the sequence, lengths on and off the 64-token tile boundary, several
    token ranges per strip."""
    L, B, d, dtype = 2, 4, 128, torch.bfloat16
    cap = max(lens) + 3
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=cap, seed=77, outlier_channels=4)
    qr = synth.normal((L, B, Hq, w, d), 78, dtype)
    b = ngc()
    for lists in (1, 2):
        ref = oracle.score_evict(synth.to_numpy(c.k), c.seq_off.numpy(), c.lens.numpy(), synth.to_numpy(qr), 1, lists, n_max=cap)
        dc = to_device_cache(c, cap)
        G = oracle.lists_G(lists, L, Hkv)
        logits = torch.full((B, G, cap), -5.0, dtype=torch.float32, device="cuda")
        ws = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE, dc, G, cap))
        st = b.new_status()
        b.ngc_score_evict(dc, qr.cuda(), 1, lists, logits, ws=ws, status=st)
        torch.cuda.synchronize()
        assert status_value(st) == 0
        got = logits.cpu().numpy().astype(np.float64)
        live = ~np.isnan(ref)
        assert np.all(got[~live] == -5.0)
        for bb in range(B):
            for g in range(G):
                m = live[bb, g]
                assert np.max(np.abs(got[bb, g][m] - ref[bb, g][m])) <= 2e-2 * ref[bb, g][m].max()
                assert abs(got[bb, g][m].sum() - 1.0) <= 1e-3          # psi is a mean of probability rows


# ------------------------------------------------------------------ lists of at most 32 units (warp-per-list kernels)

@pytest.mark.parametrize("B,G,n_max", [(37, 28, 16), (19, 28, 22), (5, 3, 32), (9, 1, 2), (64, 56, 8)])
def test_tiny_lists_sample_and_logprob(B, G, n_max):
    """The paper's own list sizes (block-level eviction: 16-22 units per layer): sampling bit-exact,
    log-prob within 1e-3 (fp64: far inside), ragged n, protected prefixes, K = n and K = P included."""
    rng = np.random.default_rng(B * 1000 + n_max)
    logits = synth.make_logits(B, G, n_max, seed=n_max + 5, std=1.3).numpy()
    logits[0, 0, : min(4, n_max)] = 0.5                                     # ties
    n = rng.integers(1, n_max + 1, B).astype(np.int32)
    n[0] = n_max
    P = np.array([rng.integers(0, x // 3 + 1) for x in n], np.int32)
    K = np.array([rng.integers(p, x + 1) for p, x in zip(P, n)], np.int32)
    K[0] = max(P[0], n_max // 2)
    if B > 2:
        K[1] = n[1]
        K[2] = P[2]
    k_max = int(K.max()) + 2
    for greedy in (0, 1):
        ref = oracle.sample_evict(logits, n, P, K, k_max, seed=5, rnd=9, greedy=greedy, list_base=3)
        got = gpu_sample(logits, n, P, K, k_max, seed=5, rnd=9, greedy=greedy, list_base=3)
        assert got[3] == 0 and not ref[3].any()
        for i in range(3):
            assert np.array_equal(got[i], ref[i])
        lp_ref, rc = oracle.evict_logprob(logits, n, P, K, ref[0])
        lp, st = gpu_logprob(logits, n, P, K, ref[0])
        assert rc == 0 and st == 0
        assert np.max(np.abs(lp - lp_ref)) <= TOL_LOGP and np.max(np.abs(lp - lp_ref)) <= 1e-9


def test_tiny_lists_status_paths():
    logits = synth.make_logits(4, 2, 20, seed=2).numpy()
    n = np.array([20, 12, 20, 7], np.int32)
    K = np.array([10, 6, 10, 3], np.int32)
    logits[1, 1, 4] = np.nan                                              # NaN candidate -> list blanked, status 2
    ref = oracle.sample_evict(logits, n, None, K, 10, seed=1, rnd=1)
    got = gpu_sample(logits, n, None, K, 10, seed=1, rnd=1)
    assert got[3] == 2 and ref[3][1, 1] == 2
    for i in range(3):
        assert np.array_equal(got[i], ref[i])
    got = gpu_sample(logits, n, None, np.array([21, 6, 10, 3], np.int32), 21, seed=1, rnd=1)   # K > n -> status 1
    assert got[3] == 1 and np.all(got[0][0] == -1) and np.all(got[1][0] == -1) and got[2][0].sum() == 0
    # log-prob: repeated unit, out-of-range unit, NaN logit
    logits[1, 1, 4] = 0.0
    ko = oracle.sample_evict(logits, n, None, K, 10, seed=1, rnd=1)[0]
    good = oracle.evict_logprob(logits, n, None, K, ko)[0]
    bad = ko.copy()
    bad[2, 0, 1] = bad[2, 0, 0]
    lp, st = gpu_logprob(logits, n, None, K, bad)
    assert st == 3 and math.isnan(lp[0, 2, 0]) and abs(lp[0, 0, 0] - good[0, 0, 0]) < 1e-9
    bad = ko.copy()
    bad[3, 1, 2] = 7                                                      # unit 7 of a list of 7 units
    lp, st = gpu_logprob(logits, n, None, K, bad)
    assert st == 3 and math.isnan(lp[0, 3, 1])
    logits[0, 1, 3] = np.nan
    lp, st = gpu_logprob(logits, n, None, K, ko)
    assert st == 2 and math.isnan(lp[0, 0, 1]) and abs(lp[0, 1, 0] - good[0, 1, 0]) < 1e-9


# ------------------------------------------------------------------ gradient of the log-prob

TOL_GRAD = 2e-6      # fp32 output of an fp64 computation; entries are O(1)


@pytest.mark.parametrize("NB,B,G,n_max,frac", [(1, 3, 2, 700, 0.5), (3, 2, 2, 768, 1 / 3), (1, 2, 1, 4096, 0.5), (1, 1, 2, 16384, 0.5),
                                                (2, 2, 1, 40, 1.0), (2, 9, 28, 16, 0.5), (1, 7, 28, 22, 0.5), (1, 4, 1, 32, 0.25)])
def test_logprob_grad_matches_oracle(NB, B, G, n_max, frac):
    rng = np.random.default_rng(n_max + 7 * NB)
    logits = synth.make_logits(NB * B, G, n_max, seed=n_max + 1, std=1.5).numpy().reshape(NB, B, G, n_max)
    n = rng.integers(max(1, n_max // 2), n_max + 1, (NB, B)).astype(np.int32)
    P = rng.integers(0, 3, (NB, B)).astype(np.int32)
    P = np.minimum(P, n)
    K = np.minimum(n, np.maximum(P, np.ceil(n * frac).astype(np.int32)))
    k_max = int(K.max())
    ko = np.stack([oracle.sample_evict(logits[r], n[r], P[r], K[r], k_max, seed=3, rnd=r)[0] for r in range(NB)])
    up = rng.normal(0, 1, (NB, B, G))
    ref, rc = oracle.evict_logprob_grad(logits, n, P, K, ko, grad_logp=up)
    assert rc == 0
    got, st = gpu_logprob_grad(logits, n, P, K, ko, grad_logp=up)
    assert st == 0
    assert np.max(np.abs(got - ref)) <= TOL_GRAD
    # no upstream gradient given = ones; every entry written (padding and protected units are zero)
    got1, st = gpu_logprob_grad(logits, n, P, K, ko)
    ref1, _ = oracle.evict_logprob_grad(logits, n, P, K, ko)
    assert st == 0 and np.max(np.abs(got1 - ref1)) <= TOL_GRAD
    assert np.max(np.abs(got1.sum(-1))) <= 1e-4                     # shift invariance of Eq. (1)


@pytest.mark.parametrize("n_max", [20, 300])
def test_logprob_grad_bad_lists(n_max):
    logits = synth.make_logits(3, 1, n_max, seed=1).numpy()
    n = np.array([n_max, n_max - 3, n_max], np.int32)
    K = np.array([n_max // 2, n_max // 4, n_max // 2], np.int32)
    ko = oracle.sample_evict(logits, n, None, K, int(K.max()), seed=8, rnd=0)[0]
    good = oracle.evict_logprob_grad(logits, n, None, K, ko)[0]
    bad = ko.copy()
    bad[1, 0, 1] = bad[1, 0, 0]                                      # repeated unit
    got, st = gpu_logprob_grad(logits, n, None, K, bad)
    assert st == 3 and np.isnan(got[0, 1, 0]).all() and np.max(np.abs(got[0, 0] - good[0, 0])) <= TOL_GRAD
    got, st = gpu_logprob_grad(logits, n, None, np.array([n_max + 1, K[1], K[2]], np.int32), ko)
    assert st == 1 and np.isnan(got[0, 0, 0]).all()
    logits[2, 0, 5] = np.nan
    got, st = gpu_logprob_grad(logits, n, None, K, ko)
    assert st == 2 and np.isnan(got[0, 2, 0]).all() and np.max(np.abs(got[0, 1] - good[0, 1])) <= TOL_GRAD


# ------------------------------------------------------------------ many short strips

@pytest.mark.parametrize("Hq,Hkv", [(12, 2), (28, 4), (8, 8)])
def test_decode_many_short_strips(Hq, Hkv):
    """Hundreds of short strips (the paper's own cache sizes): ragged lengths incl. empty and single-token
    sequences, lengths on tile borders, two appending steps, every sequence checked."""
    b = ngc()
    L, B, d, dtype = 4, 230, 128, torch.bfloat16
    rng = np.random.default_rng(Hq)
    lens = rng.integers(0, 700, B).astype(np.int32)
    lens[:8] = [0, 1, 63, 64, 65, 127, 128, 699]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=702, seed=21, outlier_channels=4)
    dc = to_device_cache(c, 702)
    k_ref, v_ref = synth.to_numpy(c.k).copy(), synth.to_numpy(c.v).copy()
    so, o_lens = c.seq_off.numpy(), lens.copy()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, dc))
    st = b.new_status()
    out = torch.full((L, B, Hq, d), 7.0, dtype=torch.float32, device="cuda")
    for s in range(2):
        q = synth.make_queries(L, B, Hq, d, dtype, seed=30 + s)
        nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=40 + 2 * s)
        b.ngc_decode_attn_ragged(dc, q.cuda(), out, nk.cuda(), nv.cuda(), ws=ws, status=st)
        ref, rc = oracle.decode_attn(k_ref, v_ref, so, o_lens, synth.to_numpy(q), synth.to_numpy(nk), synth.to_numpy(nv))
        assert rc == 0
        assert max_rel_err_per_vector(out.cpu().numpy().astype(np.float64), ref) <= TOL_ATTN_BF16
    torch.cuda.synchronize()
    assert status_value(st) == 0 and np.array_equal(dc.lens.cpu().numpy(), o_lens)
    kg, vg = synth.to_numpy(dc.k), synth.to_numpy(dc.v)
    for bb in range(B):
        sl = slice(so[bb], so[bb] + o_lens[bb])
        assert np.array_equal(kg[:, :, sl], k_ref[:, :, sl]) and np.array_equal(vg[:, :, sl], v_ref[:, :, sl])
    # read-only call (no append): the empty sequences give zeros
    dc.lens.copy_(torch.as_tensor(lens))
    q = synth.make_queries(L, B, Hq, d, dtype, seed=50)
    b.ngc_decode_attn_ragged(dc, q.cuda(), out, ws=ws, status=st)
    ref, _ = oracle.decode_attn(k_ref, v_ref, so, lens.copy(), synth.to_numpy(q))
    got = out.cpu().numpy().astype(np.float64)
    assert max_rel_err_per_vector(got, ref) <= TOL_ATTN_BF16 and np.all(got[:, 0] == 0.0)


def test_decode_on_a_second_device_after_the_first():
    """The kernels' opt-in to large dynamic shared memory is stored per device: a process that drives GPU 0 and then
    GPU 1 must get the same result on both (needs two devices; one-device boxes skip)."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two CUDA devices")
    b = ngc()
    L, B, Hq, Hkv, d, T = 2, 3, 12, 2, 128, 500
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.bfloat16, [T, 77, 300], capacity=T + 1, seed=21, outlier_channels=4)
    q = synth.make_queries(L, B, Hq, d, torch.bfloat16, seed=22)
    outs = []
    for dev in (0, 1):
        with torch.cuda.device(dev):
            dn = f"cuda:{dev}"
            dc = b.NgcCache(c.k.to(dn), c.v.to(dn), c.seq_off.to(dn), c.lens.to(dn), Hq, T)
            out = torch.zeros((L, B, Hq, d), dtype=torch.float32, device=dn)
            st = b.new_status(dn)
            ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, dc), dn)
            b.ngc_decode_attn_ragged(dc, q.to(dn), out, ws=ws, status=st)
            qr = synth.normal((L, B, Hq, 5, d), 23, torch.bfloat16).to(dn)
            lg = torch.zeros((B, 1, T), dtype=torch.float32, device=dn)
            ws2 = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE, dc, 1, T), dn)
            b.ngc_score_evict(dc, qr, 1, b.LISTS_SHARED, lg, ws=ws2, status=st)
            torch.cuda.synchronize(dev)
            assert int(st.item()) == 0
            outs.append((out.cpu(), lg.cpu()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_bounded_wait_runs_out_and_reports_timeout():
    """The kernels wait for their TMA data with a time limit.  A wait that nothing ever completes (an mbarrier no one
    arrives on, limit 2 ms) must end in NGC_DEV_TIMEOUT with a normal return, and the context must stay usable."""
    b = ngc()
    st = b.new_status()
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    b.ngc_selftest_bounded_wait(2000, st, waited)
    torch.cuda.synchronize()
    assert status_value(st) == 6                      # NGC_DEV_TIMEOUT
    assert 2_000_000 <= int(waited.item()) < 200_000_000
    # the device still works: an ordinary call behind it
    c = synth.make_cache(1, 1, 4, 4, 64, torch.float32, [9], capacity=9, seed=1)
    q = synth.make_queries(1, 1, 4, 64, torch.float32, seed=2)
    dc, got, st2 = run_decode(c, q)
    _, _, _, ref, rc = oracle_decode(c, q)
    assert st2 == 0 and rc == 0 and np.max(np.abs(got - ref)) <= TOL_ATTN_F32
    with pytest.raises(b.NgcError):
        b.ngc_selftest_bounded_wait(10_000_000, st)   # limits beyond 100 ms are refused
