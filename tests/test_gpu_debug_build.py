"""The stand-in for a memory checker, in two parts.

(1) The bounds-checking build of the library (``build.py --debug``): its kernels check every index
they compute right before using it and report a violation through the device status word instead
of touching memory.  A spread of the small parity cases of the other GPU test files is rerun on
that build; they pass only if results AND status are what they are on the normal build, i.e. no
check fired.

(2) Canaries: the K/V buffers sit between guard planes, every sequence has spare rows behind its
live part, and the small output arrays carry guard elements behind their end, all filled with a
pattern.  After compaction, appends, paged eviction and the scoring / sampling calls everything
the call had no business writing must still hold the pattern.
"""
import numpy as np
import pytest
import torch

import oracle
import test_gpu_decode_random as t_rand
import test_gpu_list_lens as t_lens
import test_gpu_paged as t_paged
import test_gpu_parity as t_par
import test_gpu_replay as t_replay
import test_gpu_replay_attn as t_rattn
import test_gpu_score_backward as t_sbwd
from helpers import ngc, status_value
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu

bf16, f32 = torch.bfloat16, torch.float32

CASES = [
    (t_par.test_sample_bit_exact, (3, 2, 100, 1.0)),
    (t_par.test_sample_bit_exact, (2, 3, 4096, 1.4142)),
    (t_par.test_sample_bit_exact, (2, 2, 16384, 1.0)),
    (t_par.test_sample_long_lists_with_ties_around_the_selection_threshold, ("quantised",)),
    (t_par.test_sample_edge_cases_and_status, ()),
    (t_par.test_tiny_lists_sample_and_logprob, (19, 28, 22)),
    (t_par.test_logprob_matches_oracle, (4, 2, 3, 768, 1 / 3)),
    (t_par.test_logprob_grad_matches_oracle, (3, 2, 2, 768, 1 / 3)),
    (t_par.test_compact_bit_exact, (bf16, 128, 0)),
    (t_par.test_compact_bit_exact, (f32, 64, 2)),
    (t_par.test_compact_bit_exact, (bf16, 64, 1)),
    (t_par.test_compact_blocks_ragged_and_corrupt_lists, ()),
    (t_par.test_compact_per_list_disagreement_is_reported, ()),
    (t_par.test_compact_sequence_with_one_corrupt_list_is_left_whole, ()),
    (t_par.test_decode_matches_oracle, (f32, 64, 4, 4, t_par.TOL_ATTN_F32)),
    (t_par.test_decode_matches_oracle, (bf16, 128, 12, 2, t_par.TOL_ATTN_BF16)),
    (t_par.test_decode_matches_oracle, (bf16, 128, 16, 1, t_par.TOL_ATTN_BF16)),
    (t_par.test_decode_matches_oracle, (bf16, 128, 40, 2, t_par.TOL_ATTN_BF16)),
    (t_par.test_decode_append_and_layer_ranges, (f32, 64, 4, 4)),
    (t_par.test_decode_append_and_layer_ranges, (bf16, 128, 12, 2)),
    (t_par.test_decode_full_strip_is_reported_and_skipped, ()),
    (t_par.test_decode_bf16_output_and_token_splits, ()),
    (t_par.test_decode_many_short_strips, (28, 4)),
    (t_par.test_score_matches_oracle, (bf16, 128, 12, 2, 1, 32)),
    (t_par.test_score_matches_oracle, (f32, 64, 4, 4, 2, 1)),
    (t_par.test_score_window_sizes_and_ragged_lengths, (28, 4, 5, [4, 5, 6, 3000])),
    (t_rand.test_decode_random_shapes, (3,)),
    (t_rand.test_paged_decode_random_shapes, (2,)),
    (t_paged.test_paged_evict_and_decode_match_oracle, (32, 1, [317, 93, 29, 637])),
    (t_paged.test_paged_full_sequence_and_bad_list_are_reported, ()),
    (t_paged.test_paged_lists_with_their_own_lengths, ()),
    (t_lens.test_per_list_lengths_through_three_rounds, (1,)),
    (t_replay.test_replay_visibility_matches_oracle, (5, 2, 3, 4, 5, 70)),
    (t_replay.test_replay_visibility_figure_and_failures, ()),
    (t_rattn.test_replay_attn_matches_oracle, (2, 4, 3, 30, 200, None)),
    (t_rattn.test_replay_attn_matches_oracle, (1, 32, 2, 100, 300, 1)),
    (t_sbwd.test_score_backward_matches_oracle, (12, 2, 5, 1, 32, 0)),
]


@pytest.fixture(scope="module")
def debug_library():
    from paper_2604_18002_b200 import binding, build
    path = build.build(debug=True)
    with binding.use_library(path):
        yield path


@pytest.mark.parametrize("case", range(len(CASES)), ids=[f"{f.__name__}-{i}" for i, (f, _) in enumerate(CASES)])
def test_small_parity_case_on_the_bounds_checking_build(case, debug_library):
    fn, args = CASES[case]
    fn(*args)


def test_bounds_checking_build_is_a_different_library_with_the_same_exports(debug_library):
    b = ngc()
    assert debug_library.endswith("libngc_b200_debug.so") and b.lib._name == debug_library
    for sym in b.EXPORTS:
        assert hasattr(b.lib, sym)


# ------------------------------------------------------------------ canaries

PATTERN = 0x7B7B          # bf16 bit pattern of the guard rows (a large finite number: it would show in any sum)


def guarded_cache(L, B, Hq, Hkv, d, lens, cap, seed):
    """A bf16 cache whose K and V sit between two guard planes; rows at and beyond lens[b] hold the pattern."""
    b = ngc()
    c = synth.make_cache(L, B, Hq, Hkv, d, bf16, lens, capacity=cap, seed=seed, outlier_channels=4)
    so = c.seq_off.numpy()
    R = int(so[-1])
    planes = L * Hkv
    bufs = []
    for src in (c.k, c.v):
        flat = torch.full((planes + 2, R, d), PATTERN, dtype=torch.int16)
        flat[1:-1] = src.view(torch.int16).reshape(planes, R, d)
        for bb in range(B):
            flat[1:-1, so[bb] + lens[bb]:so[bb + 1]] = PATTERN
        bufs.append(flat.cuda())
    k = bufs[0][1:-1].view(torch.bfloat16).view(L, Hkv, R, d)
    v = bufs[1][1:-1].view(torch.bfloat16).view(L, Hkv, R, d)
    host = synth.Cache(k.cpu(), v.cpu(), c.seq_off, c.lens, L, B, Hq, Hkv, d)      # what the oracle sees
    dc = b.NgcCache(k, v, c.seq_off.cuda(), c.lens.clone().cuda(), Hq, int(max(cap) if hasattr(cap, "__len__") else cap))
    return host, dc, bufs, so


def planes_i16(dc):
    L, Hkv, R, d = dc.k.shape
    return dc.k.view(torch.int16).cpu().numpy(), dc.v.view(torch.int16).cpu().numpy()


def assert_guards(bufs):
    for buf in bufs:
        assert bool((buf[0] == PATTERN).all()) and bool((buf[-1] == PATTERN).all()), "a guard plane was written"


def guarded(shape, dtype, extra=64):
    """Device array with `extra` guard elements behind its end; returns (array view, whole buffer, fill)."""
    n = int(np.prod(shape))
    fill = -12345 if dtype in (torch.int32, torch.int16) else 777.0
    whole = torch.full((n + extra,), fill, dtype=dtype, device="cuda")
    return whole[:n].view(shape), whole, fill


@pytest.mark.parametrize("lists,block", [(0, 1), (1, 32), (2, 1)])
def test_canaries_survive_compaction_and_appends(lists, block):
    b = ngc()
    L, B, Hq, Hkv, d, steps = 2, 3, 12, 2, 128, 5
    lens = [700, 33, 257]
    cap = [l + steps + 2 for l in lens]                       # 2 spare rows behind everything a sequence will ever hold
    host, dc, bufs, so = guarded_cache(L, B, Hq, Hkv, d, lens, cap, seed=31)
    G = oracle.lists_G(lists, L, Hkv)
    units = [(l + block - 1) // block for l in lens]
    budget = np.array([max(1, u // 2) for u in units], np.int32)
    n_max, k_max = max(units), int(budget.max())
    logits = synth.make_logits(B, G, n_max, seed=32).numpy()
    if block > 1:
        logits[:, :, :] = np.where(np.arange(n_max)[None, None] == np.array(units)[:, None, None] - 1, -50.0, logits)  # drop the short last unit everywhere
    ko, ks, _, st0 = oracle.sample_evict(logits, units, None, budget, k_max, seed=5, rnd=0)
    assert not st0.any()
    kc, vc, nl, rc = oracle.compact_kv(synth.to_numpy(host.k), synth.to_numpy(host.v), so, np.array(lens, np.int32), ks, budget, lists, block)
    assert rc == 0
    before_k, before_v = planes_i16(dc)
    st = b.new_status()
    b.ngc_compact_kv(dc, torch.as_tensor(ks).cuda(), torch.as_tensor(budget).cuda(), lists, block, status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 0 and np.array_equal(dc.lens.cpu().numpy(), nl)
    after_k, after_v = planes_i16(dc)
    for bb in range(B):
        live = slice(so[bb], so[bb] + nl[bb])
        rest = slice(so[bb] + nl[bb], so[bb + 1])
        assert np.array_equal(after_k[:, :, live].view(np.uint16), kc[:, :, live]) and np.array_equal(after_v[:, :, live].view(np.uint16), vc[:, :, live])
        # compaction writes destination rows only: everything at and beyond the new length is as it was
        assert np.array_equal(after_k[:, :, rest], before_k[:, :, rest]) and np.array_equal(after_v[:, :, rest], before_v[:, :, rest])
    assert_guards(bufs)
    # appends: exactly one row per strip and step
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, dc))
    out, out_whole, out_fill = guarded((L, B, Hq, d), torch.float32)
    for s in range(steps):
        q = synth.make_queries(L, B, Hq, d, bf16, seed=40 + s).cuda()
        nk, nv = synth.make_new_kv(L, B, Hkv, d, bf16, seed=60 + 2 * s)
        b.ngc_decode_attn_ragged(dc, q, out, nk.cuda(), nv.cuda(), ws=ws, status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 0
    end_k, end_v = planes_i16(dc)
    for bb in range(B):
        tail = slice(so[bb] + nl[bb] + steps, so[bb + 1])
        head = slice(so[bb], so[bb] + nl[bb])
        assert np.array_equal(end_k[:, :, tail], after_k[:, :, tail]) and np.array_equal(end_v[:, :, tail], after_v[:, :, tail])
        assert np.array_equal(end_k[:, :, head], after_k[:, :, head]) and np.array_equal(end_v[:, :, head], after_v[:, :, head])
    assert_guards(bufs)
    assert bool((out_whole[out.numel():] == out_fill).all())


def test_canaries_survive_score_sample_and_logprob():
    b = ngc()
    L, B, Hq, Hkv, d, T, w = 2, 3, 12, 2, 128, 600, 5
    lens = [T, 77, 300]
    host, dc, bufs, so = guarded_cache(L, B, Hq, Hkv, d, lens, [T + 2] * B, seed=33)
    G, n_max, k_max = L, T + 2, T // 2                      # n_max covers the row capacity
    logits, lg_whole, lg_fill = guarded((B, G, n_max), torch.float32)
    qr = synth.normal((L, B, Hq, w, d), 34, bf16).cuda()
    st = b.new_status()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE, dc, G, n_max))
    n_out, n_whole, n_fill = guarded((B,), torch.int32)
    b.ngc_score_evict(dc, qr, 1, b.LISTS_PER_LAYER, logits, ws=ws, status=st, n_units_out=n_out)
    ko, ko_whole, i_fill = guarded((B, G, k_max), torch.int32)
    ks, ks_whole, _ = guarded((B, G, k_max), torch.int32)
    km, km_whole, _ = guarded((B, G, n_max), torch.int16)
    lp, lp_whole, lp_fill = guarded((1, B, G), torch.float64)
    budget = torch.as_tensor(np.array([l // 2 for l in lens], np.int32)).cuda()
    b.ngc_sample_evict(logits, n_out, None, budget, 3, 0, ko, ks, None, status=st)
    b.ngc_evict_logprob(logits, n_out, None, budget, ko, lp, status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 0 and list(n_out.cpu().numpy()) == lens
    lg = logits.cpu().numpy()
    for bb in range(B):
        assert np.all(lg[bb, :, lens[bb]:] == lg_fill)                     # units the sequence does not have: untouched
        assert abs(lg[bb, :, :lens[bb]].sum() - G) <= 1e-2                 # every layer's scores sum to one
    for whole, view, fill in ((lg_whole, logits, lg_fill), (n_whole, n_out, n_fill), (ko_whole, ko, i_fill), (ks_whole, ks, i_fill),
                              (lp_whole, lp, lp_fill)):
        assert bool((whole[view.numel():] == fill).all()), "a guard element behind an output array was written"
    k_now, v_now = planes_i16(dc)
    assert np.array_equal(k_now.view(np.uint16), synth.to_numpy(host.k)) and np.array_equal(v_now.view(np.uint16), synth.to_numpy(host.v))   # read-only calls
    assert_guards(bufs)


def test_canaries_survive_paged_eviction():
    b = ngc()
    L, B, Hq, Hkv, d, page, pages_cap, lists = 2, 3, 12, 2, 128, 32, 12, 1
    lens = [300, 97, 33]
    c = synth.make_cache(L, B, Hq, Hkv, d, bf16, lens, capacity=pages_cap * page, seed=35)
    pc = t_paged.to_paged(c, page, pages_cap, lists, seed=36)
    G = L
    table, table_whole, t_fill = guarded((B, G, pages_cap), torch.int32)
    table.copy_(pc.page_table)
    pc.page_table = table
    k0, v0 = pc.k.view(torch.int16).clone(), pc.v.view(torch.int16).clone()    # bit patterns: the free pages hold junk, NaNs included
    units = [(l + page - 1) // page for l in lens]
    budget = np.array([max(1, u // 2) for u in units], np.int32)
    logits = synth.make_logits(B, G, pages_cap, seed=37).numpy()
    logits[:, :, :] = np.where(np.arange(pages_cap)[None, None] == np.array(units)[:, None, None] - 1, 50.0, logits)   # every list keeps the short last page
    ko, ks, _, st0 = oracle.sample_evict(logits, units, None, budget, int(budget.max()), seed=6, rnd=0, greedy=1)
    st = b.new_status()
    b.ngc_evict_pages(pc, torch.as_tensor(ks).cuda(), torch.as_tensor(budget).cuda(), status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 0
    assert torch.equal(pc.k.view(torch.int16), k0) and torch.equal(pc.v.view(torch.int16), v0)   # eviction on a paged cache moves no K/V row
    assert bool((table_whole[table.numel():] == t_fill).all())
    rows = table.cpu().numpy()
    assert np.all(np.sort(rows, -1) == np.arange(pages_cap))               # every row is still a permutation of the pool
