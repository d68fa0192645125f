"""One cache length per (sequence, list): the paper evicts per layer in units of 32 tokens, and when a
round fires at a length that is not a multiple of the unit, a layer that keeps the short last unit
ends up with fewer tokens than one that evicts it.  Three rounds of score -> sample -> log-prob ->
compact -> decode with per-layer lists; every layer is checked against the oracle run on that layer
alone (the oracle knows one length per sequence)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import max_rel_err_per_vector, ngc, status_value
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("lists", [1, 2])
def test_per_list_lengths_through_three_rounds(lists):
    b = ngc()
    L, B, Hq, Hkv, d, dtype, block, w = 3, 3, 12, 2, 128, torch.bfloat16, 32, 5
    G = oracle.lists_G(lists, L, Hkv)
    cap = 640
    lens0 = [200, 97, 333]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens0, capacity=cap, seed=12, outlier_channels=4)
    so = c.seq_off.numpy()
    lens_d = torch.as_tensor(np.repeat(np.array(lens0, np.int32)[:, None], G, 1)).cuda().contiguous()
    dc = b.NgcCache(c.k.cuda(), c.v.cuda(), c.seq_off.cuda(), lens_d, Hq, cap, lists)
    # host mirror: one single-plane cache per list (layer, or layer and KV head), with its own lengths
    kh, vh = synth.to_numpy(c.k), synth.to_numpy(c.v)

    def plane(a, g):          # the planes list g covers, as a cache of its own
        if lists == 1:
            return np.ascontiguousarray(a[g:g + 1])
        return np.ascontiguousarray(a[g // Hkv:g // Hkv + 1, g % Hkv:g % Hkv + 1])
    Hq_g, Hkv_g = (Hq, Hkv) if lists == 1 else (Hq // Hkv, 1)
    k_ref = [plane(kh, g) for g in range(G)]
    v_ref = [plane(vh, g) for g in range(G)]
    o_lens = [np.array(lens0, np.int32) for _ in range(G)]

    def heads(t, g):          # the query heads (dim 2 of [L][B][Hq]...) feeding list g
        if lists == 1:
            return t[g:g + 1]
        l, h = g // Hkv, g % Hkv
        return t[l:l + 1, :, h * Hq_g:(h + 1) * Hq_g]

    def kv_new(t, g):         # [L][B][Hkv][d] -> the list's planes
        return t[g:g + 1] if lists == 1 else t[g // Hkv:g // Hkv + 1, :, g % Hkv:g % Hkv + 1]

    st = b.new_status()
    ws_d = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, dc))
    out = torch.zeros((L, B, Hq, d), dtype=torch.float32, device="cuda")
    n_max = cap // block
    ws_s = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE, dc, G, n_max))
    step = 0
    differed = False
    for rnd in range(3):
        for _ in range(7):
            q = synth.make_queries(L, B, Hq, d, dtype, seed=100 + step)
            nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=200 + 2 * step)
            b.ngc_decode_attn_ragged(dc, q.cuda(), out, nk.cuda(), nv.cuda(), ws=ws_d, status=st)
            got = out.cpu().numpy().astype(np.float64)
            for g in range(G):
                ref, rc = oracle.decode_attn(k_ref[g], v_ref[g], so, o_lens[g], synth.to_numpy(heads(q, g).contiguous()),
                                             synth.to_numpy(kv_new(nk, g).contiguous()), synth.to_numpy(kv_new(nv, g).contiguous()))
                assert rc == 0
                assert max_rel_err_per_vector(heads(torch.as_tensor(got), g).numpy(), ref) <= 2e-2, (rnd, g)
            step += 1
        torch.cuda.synchronize()
        assert np.array_equal(dc.lens.cpu().numpy(), np.stack(o_lens, 1))
        # scores of every list at its own length; the library itself writes -inf into the units a shorter list
        # lacks (up to the unit count of the sequence's longest list, which it also reports) and leaves the rest alone
        qr = synth.normal((L, B, Hq, w, d), 300 + rnd, dtype)
        logits = torch.full((B, G, n_max), 123.0, dtype=torch.float32, device="cuda")
        n_out = torch.full((B,), -5, dtype=torch.int32, device="cuda")
        b.ngc_score_evict(dc, qr.cuda(), block, lists, logits, ws=ws_s, status=st, n_units_out=n_out)
        lg = logits.cpu().numpy()
        units_now = np.stack([(o + block - 1) // block for o in o_lens], 1)         # [B][G]
        assert np.array_equal(n_out.cpu().numpy(), units_now.max(1))
        for g in range(G):
            ref_s = oracle.score_evict(k_ref[g], so, o_lens[g], synth.to_numpy(heads(qr, g).contiguous()), block, 0, n_max=n_max)
            live = ~np.isnan(ref_s[:, 0])
            for bb in range(B):
                assert np.all(np.isneginf(lg[bb, g, units_now[bb, g]:units_now[bb].max()]))
                assert np.all(lg[bb, g, units_now[bb].max():] == 123.0)
            for bb in range(B):
                m = live[bb]
                assert np.max(np.abs(lg[bb, g][m] - ref_s[bb, 0][m])) <= 2e-2 * ref_s[bb, 0][m].max()
        # the draw: n = the largest unit count of the sequence's lists; missing units carry -inf and are never drawn
        units = np.stack([(o + block - 1) // block for o in o_lens], 1)             # [B][G]
        n_b = units.max(1).astype(np.int32)
        budget = np.maximum(1, units.min(1) // 2).astype(np.int32)
        k_max = int(budget.max())
        lg_syn = synth.make_logits(B, G, n_max, seed=400 + rnd).numpy()
        for bb in range(B):
            for g in range(G):
                lg_syn[bb, g, units[bb, g]:] = -np.inf
        r_ko, r_ks, _, rst = oracle.sample_evict(lg_syn, n_b, None, budget, k_max, seed=7, rnd=rnd)
        assert not rst.any()
        ko = torch.empty((B, G, k_max), dtype=torch.int32, device="cuda")
        ks = torch.empty_like(ko)
        lp = torch.empty((1, B, G), dtype=torch.float64, device="cuda")
        lg_t, n_t, k_t = torch.as_tensor(lg_syn).cuda(), torch.as_tensor(n_b).cuda(), torch.as_tensor(budget).cuda()
        b.ngc_sample_evict(lg_t, n_t, None, k_t, 7, rnd, ko, ks, None, status=st)
        b.ngc_evict_logprob(lg_t, n_t, None, k_t, ko, lp, status=st)
        assert np.array_equal(ko.cpu().numpy(), r_ko) and np.array_equal(ks.cpu().numpy(), r_ks)
        lp_ref, rc = oracle.evict_logprob(lg_syn, n_b, None, budget, r_ko)
        assert rc == 0 and np.max(np.abs(lp.cpu().numpy() - lp_ref)) <= 1e-3
        # physical eviction: every list ends at its own length
        b.ngc_compact_kv(dc, ks, k_t, lists, block, status=st)
        torch.cuda.synchronize()
        assert status_value(st) == 0
        kg, vg = synth.to_numpy(dc.k), synth.to_numpy(dc.v)
        for g in range(G):
            k_ref[g], v_ref[g], nl, rc = oracle.compact_kv(k_ref[g], v_ref[g], so, o_lens[g], r_ks[:, g:g + 1], budget, 0, block)
            assert rc == 0
            o_lens[g] = nl.copy()
            for bb in range(B):
                sl = slice(so[bb], so[bb] + nl[bb])
                assert np.array_equal(plane(kg, g)[:, :, sl], k_ref[g][:, :, sl]) and np.array_equal(plane(vg, g)[:, :, sl], v_ref[g][:, :, sl])
        got_lens = dc.lens.cpu().numpy()
        assert np.array_equal(got_lens, np.stack(o_lens, 1))
        differed = differed or bool((got_lens.max(1) != got_lens.min(1)).any())
    assert differed          # the scenario really produced lists of different lengths


def test_one_length_per_sequence_still_reports_disagreement():
    b = ngc()
    L, B, Hq, Hkv, d, dtype, block = 2, 1, 4, 2, 128, torch.bfloat16, 32
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, [100], capacity=128, seed=1)
    dc = b.NgcCache(c.k.cuda(), c.v.cuda(), c.seq_off.cuda(), c.lens.cuda(), Hq, 128)
    ks = torch.tensor([[[0, 3], [1, 2]]], dtype=torch.int32).cuda()           # layer 0 keeps the short last unit, layer 1 does not
    st = b.new_status()
    b.ngc_compact_kv(dc, ks, torch.tensor([2], dtype=torch.int32).cuda(), 1, block, status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 5 and int(dc.lens.item()) == 100
    assert torch.equal(dc.k.cpu(), c.k) and torch.equal(dc.v.cpu(), c.v)      # nothing moved
    with pytest.raises(b.NgcError):                                           # a length per layer cannot serve per-head lists
        dl = b.NgcCache(dc.k, dc.v, dc.seq_off, torch.zeros((1, 2), dtype=torch.int32, device="cuda"), Hq, 128, 1)
        b.ngc_compact_kv(dl, ks, torch.tensor([2], dtype=torch.int32).cuda(), 2, block, status=st)
