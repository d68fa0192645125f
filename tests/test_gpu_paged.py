"""Paged variant of the cache (one eviction unit = one page): eviction edits the page table,
decode reads through it.  Checked against the same CPU oracle as the contiguous layout: the
logical cache (pages gathered in table order) must equal the oracle's compacted cache bit for
bit, attention within 2e-2 relative, page-table rows must stay permutations."""
import numpy as np
import pytest
import torch

import oracle
from helpers import max_rel_err_per_vector, ngc, status_value
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu


def list_of(lists, l, h, Hkv):
    return 0 if lists == 0 else (l if lists == 1 else l * Hkv + h)


def to_paged(c, page, pages_cap, lists, seed):
    """Scatter a contiguous host cache into page pools behind random page tables."""
    b = ngc()
    L, Hkv, R, d = c.k.shape
    B = c.B
    G = oracle.lists_G(lists, L, Hkv)
    rng = np.random.default_rng(seed)
    table = np.stack([np.stack([rng.permutation(pages_cap) for _ in range(G)]) for _ in range(B)]).astype(np.int32)
    kp = torch.zeros((L, Hkv, B * pages_cap, page, d), dtype=c.k.dtype)
    vp = torch.zeros_like(kp)
    # free pages hold junk, as a real pool would
    kp.view(torch.int16).random_(-30000, 30000)
    vp.view(torch.int16).random_(-30000, 30000)
    so = c.seq_off.numpy()
    lens = c.lens.numpy()
    for bb in range(B):
        for l in range(L):
            for h in range(Hkv):
                row = table[bb, list_of(lists, l, h, Hkv)]
                for j in range((lens[bb] + page - 1) // page):
                    n = min(page, lens[bb] - j * page)
                    kp[l, h, bb * pages_cap + row[j], :n] = c.k[l, h, so[bb] + j * page: so[bb] + j * page + n]
                    vp[l, h, bb * pages_cap + row[j], :n] = c.v[l, h, so[bb] + j * page: so[bb] + j * page + n]
    return b.NgcPagedCache(kp.cuda(), vp.cuda(), torch.as_tensor(table).cuda(), c.lens.clone().cuda(), c.Hq, lists)


def logical(pc, bb, lens_b):
    """Host copy of sequence bb's alive rows, gathered through the page table: [L][Hkv][len][d]."""
    L, Hkv, _, page, d = pc.k.shape
    pages_cap = pc.page_table.shape[2]
    table = pc.page_table.cpu().numpy()
    k = synth.to_numpy(pc.k)
    v = synth.to_numpy(pc.v)
    ko = np.zeros((L, Hkv, lens_b, d), k.dtype)
    vo = np.zeros_like(ko)
    for l in range(L):
        for h in range(Hkv):
            row = table[bb, list_of(pc.lists, l, h, Hkv)]
            for j in range((lens_b + page - 1) // page):
                n = min(page, lens_b - j * page)
                ko[l, h, j * page: j * page + n] = k[l, h, bb * pages_cap + row[j], :n]
                vo[l, h, j * page: j * page + n] = v[l, h, bb * pages_cap + row[j], :n]
    return ko, vo


def check_logical_equals(pc, k_ref, v_ref, so, lens):
    for bb in range(len(lens)):
        kl, vl = logical(pc, bb, int(lens[bb]))
        assert np.array_equal(kl, k_ref[:, :, so[bb]: so[bb] + lens[bb]])
        assert np.array_equal(vl, v_ref[:, :, so[bb]: so[bb] + lens[bb]])


@pytest.mark.parametrize("page,lists,lens", [(64, 0, [300, 129, 64, 1]), (32, 0, [300, 97, 32, 640]), (32, 1, [317, 93, 29, 637]),
                                             (64, 2, [317, 125, 61, 637]), (32, 2, [349, 701, 61, 29])])
def test_paged_evict_and_decode_match_oracle(page, lists, lens):
    b = ngc()
    L, B, Hq, Hkv, d, dtype = 2, 4, 12, 2, 128, torch.bfloat16
    pages_cap = 24
    cap = pages_cap * page
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=cap, seed=3, outlier_channels=4)
    pc = to_paged(c, page, pages_cap, lists, seed=5)
    so = c.seq_off.numpy()
    k_ref, v_ref = synth.to_numpy(c.k).copy(), synth.to_numpy(c.v).copy()
    o_lens = c.lens.numpy().copy()
    G = oracle.lists_G(lists, L, Hkv)
    st = b.new_status()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, pc.as_contiguous_desc()))
    out = torch.empty((L, B, Hq, d), dtype=torch.float32, device="cuda")

    def decode_steps(n, seed0):
        nonlocal o_lens
        for s in range(n):
            q = synth.make_queries(L, B, Hq, d, dtype, seed=seed0 + s)
            nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=seed0 + 100 + 2 * s)
            b.ngc_decode_attn_paged(pc, q.cuda(), out, nk.cuda(), nv.cuda(), ws=ws, status=st)
            ref, rc = oracle.decode_attn(k_ref, v_ref, so, o_lens, synth.to_numpy(q), synth.to_numpy(nk), synth.to_numpy(nv))
            assert rc == 0
            assert max_rel_err_per_vector(out.cpu().numpy().astype(np.float64), ref) <= 2e-2
        torch.cuda.synchronize()
        assert status_value(st) == 0
        assert np.array_equal(pc.lens.cpu().numpy(), o_lens)
        check_logical_equals(pc, k_ref, v_ref, so, o_lens)

    # attention without append first (read-only), then a few appending steps that cross page borders
    q = synth.make_queries(L, B, Hq, d, dtype, seed=1)
    b.ngc_decode_attn_paged(pc, q.cuda(), out, ws=ws, status=st)
    ref, _ = oracle.decode_attn(k_ref, v_ref, so, o_lens.copy(), synth.to_numpy(q), None, None)
    assert max_rel_err_per_vector(out.cpu().numpy().astype(np.float64), ref) <= 2e-2
    decode_steps(3, 10)

    # scores through the page table against the oracle's scores of the contiguous cache (units = pages)
    w = 5
    qr = synth.normal((L, B, Hq, w, d), 77, dtype)
    ref_s = oracle.score_evict(k_ref, so, o_lens, synth.to_numpy(qr), page, lists, n_max=pages_cap)
    lg = torch.full((B, G, pages_cap), -5.0, dtype=torch.float32, device="cuda")
    ws_s = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE, pc.as_contiguous_desc(), G, pages_cap))
    b.ngc_score_evict_paged(pc, qr.cuda(), lg, ws=ws_s, status=st)
    torch.cuda.synchronize()
    got_s = lg.cpu().numpy().astype(np.float64)
    live = ~np.isnan(ref_s)
    assert status_value(st) == 0 and np.all(got_s[~live] == -5.0)
    for bb in range(B):
        for g in range(G):
            m = live[bb, g]
            assert np.max(np.abs(got_s[bb, g][m] - ref_s[bb, g][m])) <= 2e-2 * ref_s[bb, g][m].max()

    # one eviction round: units are pages; keep about half
    n_units = (o_lens + page - 1) // page
    budget = np.maximum(1, (n_units + 1) // 2).astype(np.int32)
    if lists != 0:
        assert not (o_lens % page).any()      # several lists per sequence: whole pages, so that they keep equal token counts
    logits = synth.make_logits(B, G, int(n_units.max()), seed=9).numpy()
    ko, ks, _, rst = oracle.sample_evict(logits, n_units.astype(np.int32), None, budget, int(budget.max()), seed=2, rnd=0)
    assert not rst.any()
    k2, v2, nl, rc = oracle.compact_kv(k_ref, v_ref, so, o_lens, ks, budget, lists, page)
    table_before = pc.page_table.cpu().numpy().copy()
    b.ngc_evict_pages(pc, torch.as_tensor(ks).cuda(), torch.as_tensor(budget).cuda(), status=st)
    torch.cuda.synchronize()
    assert rc == 0 and status_value(st) == 0
    assert np.array_equal(pc.lens.cpu().numpy(), nl)
    table = pc.page_table.cpu().numpy()
    assert np.array_equal(np.sort(table, -1), np.sort(table_before, -1))          # rows are still permutations
    for bb in range(B):
        for g in range(G):
            assert np.array_equal(table[bb, g, : budget[bb]], table_before[bb, g][ks[bb, g, : budget[bb]]])
    k_ref, v_ref, o_lens = k2, v2, nl.copy()
    check_logical_equals(pc, k_ref, v_ref, so, o_lens)
    decode_steps(page + 2, 50)       # refills the partly filled page, then takes free pages


def test_paged_full_sequence_and_bad_list_are_reported():
    b = ngc()
    L, B, Hq, Hkv, d, dtype, page, pages_cap = 1, 2, 12, 2, 128, torch.bfloat16, 32, 4
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, [128, 40], capacity=128, seed=1)
    pc = to_paged(c, page, pages_cap, 0, seed=2)
    st = b.new_status()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, pc.as_contiguous_desc()))
    out = torch.full((L, B, Hq, d), 5.0, dtype=torch.float32, device="cuda")
    q = synth.make_queries(L, B, Hq, d, dtype, seed=1)
    nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=2)
    b.ngc_decode_attn_paged(pc, q.cuda(), out, nk.cuda(), nv.cuda(), ws=ws, status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 4                                          # sequence 0 has no room for the new row
    assert np.array_equal(pc.lens.cpu().numpy(), [128, 41]) and float(out[0, 0].abs().max()) == 0.0
    st.zero_()
    table_before = pc.page_table.cpu().numpy().copy()
    ks = torch.tensor([[[0, 2]], [[1, 1]]], dtype=torch.int32).cuda()     # second list repeats a page
    b.ngc_evict_pages(pc, ks, torch.tensor([2, 2], dtype=torch.int32).cuda(), status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 3
    table = pc.page_table.cpu().numpy()
    assert np.array_equal(table[1], table_before[1]) and np.array_equal(pc.lens.cpu().numpy(), [64, 41])
    assert np.array_equal(table[0, 0, :2], table_before[0, 0][[0, 2]])


def test_paged_lists_with_their_own_lengths():
    """Per-layer lists on a paged cache with a partly filled last page: layers that keep it and layers
    that evict it end at different lengths (lens [B][G]); decode and a second round follow, every layer
    checked against the oracle run on that layer alone."""
    b = ngc()
    L, B, Hq, Hkv, d, dtype, page, pages_cap, lists = 3, 2, 12, 2, 128, torch.bfloat16, 32, 16, 1
    cap = pages_cap * page
    lens0 = [205, 77]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens0, capacity=cap, seed=21, outlier_channels=4)
    pc = to_paged(c, page, pages_cap, lists, seed=22)
    pc.lens = torch.as_tensor(np.repeat(np.array(lens0, np.int32)[:, None], L, 1)).cuda().contiguous()
    so = c.seq_off.numpy()
    kh, vh = synth.to_numpy(c.k), synth.to_numpy(c.v)
    k_ref = [np.ascontiguousarray(kh[l:l + 1]) for l in range(L)]
    v_ref = [np.ascontiguousarray(vh[l:l + 1]) for l in range(L)]
    o_lens = [np.array(lens0, np.int32) for _ in range(L)]
    st = b.new_status()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, pc.as_contiguous_desc()))
    out = torch.zeros((L, B, Hq, d), dtype=torch.float32, device="cuda")
    step = 0
    for rnd in range(2):
        units = np.stack([(o + page - 1) // page for o in o_lens], 1)
        n_b, budget = units.max(1).astype(np.int32), np.maximum(1, units.min(1) // 2).astype(np.int32)
        lg = synth.make_logits(B, L, pages_cap, seed=30 + rnd).numpy()
        for bb in range(B):
            for l in range(L):
                lg[bb, l, units[bb, l]:] = -np.inf
        r_ko, r_ks, _, rst = oracle.sample_evict(lg, n_b, None, budget, int(budget.max()), seed=3, rnd=rnd)
        assert not rst.any()
        b.ngc_evict_pages(pc, torch.as_tensor(r_ks).cuda(), torch.as_tensor(budget).cuda(), status=st)
        for l in range(L):
            k_ref[l], v_ref[l], nl, rc = oracle.compact_kv(k_ref[l], v_ref[l], so, o_lens[l], r_ks[:, l:l + 1], budget, 0, page)
            assert rc == 0
            o_lens[l] = nl.copy()
        torch.cuda.synchronize()
        assert status_value(st) == 0 and np.array_equal(pc.lens.cpu().numpy(), np.stack(o_lens, 1))
        for _ in range(5):
            q = synth.make_queries(L, B, Hq, d, dtype, seed=40 + step)
            nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=60 + 2 * step)
            b.ngc_decode_attn_paged(pc, q.cuda(), out, nk.cuda(), nv.cuda(), ws=ws, status=st)
            got = out.cpu().numpy().astype(np.float64)
            for l in range(L):
                ref, rc = oracle.decode_attn(k_ref[l], v_ref[l], so, o_lens[l], synth.to_numpy(q[l:l + 1]), synth.to_numpy(nk[l:l + 1]),
                                             synth.to_numpy(nv[l:l + 1]))
                assert rc == 0 and max_rel_err_per_vector(got[l:l + 1], ref) <= 2e-2
            step += 1
        torch.cuda.synchronize()
        assert status_value(st) == 0 and np.array_equal(pc.lens.cpu().numpy(), np.stack(o_lens, 1))
    got_lens = pc.lens.cpu().numpy()
    assert (got_lens.max(1) != got_lens.min(1)).any()
