"""ngc_replay_attn against the CPU oracle: every token of a rollout attends under its replay mask
(paper Section 4.5, Appendix A.3).  The oracle builds the paper's dense mask from the kept lists
and runs a plain masked softmax in double; the kernel gathers the kept entries instead.  Bar: 2e-2
relative per output vector (bf16 inputs, fp32 accumulation, probabilities rounded to bf16)."""
import numpy as np
import pytest
import torch

from helpers import max_rel_err_per_vector, ngc, status_value
from oracle import replay
from paper_2604_18002_b200 import synth
from test_gpu_replay import gpu_replay, random_history

pytestmark = pytest.mark.gpu


def list_of(lists, l, h, Hkv):
    return 0 if lists == 0 else (l if lists == 1 else l * Hkv + h)


def run_case(L, B, Hq, Hkv, lists, block, R, grow_lo, grow_hi, tail, seed, variant=None, key_growth=0.0):
    """``variant``: device path (None = what ngc_replay_attn runs, the tcgen05 kernel; 1 = the warp-level MMA kernel).
    ``key_growth`` > 0 scales key t by (1 + key_growth * t), so that the largest score of a row keeps growing along the
    sequence and the running maximum of the online softmax has to move many times."""
    b = ngc()
    d, dtype = 128, torch.bfloat16
    G = 1 if lists == 0 else (L if lists == 1 else L * Hkv)
    rng = np.random.default_rng(seed)
    if R:
        ks, budget, alive_before, total_before = random_history(rng, R, B, G, block, grow_lo, grow_hi)
        pos, cnt, st = gpu_replay(ks, budget, alive_before, total_before, block, int(alive_before.max()))
        assert st == 0
        T = total_before[-1] + np.asarray(tail)                   # tokens generated after the last round
    else:
        total_before = np.zeros((0, B), np.int32)
        T = np.asarray(tail)
    t_max = int(T.max())
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, T.astype(np.int32), capacity=t_max, seed=seed + 1, outlier_channels=4)
    if key_growth:
        ramp = (1.0 + key_growth * torch.arange(t_max, dtype=torch.float32)).repeat(B)[None, None, :, None]
        c.k = (c.k.float() * ramp).to(dtype)
    q = synth.normal((L, B, Hq, t_max, d), seed + 2, dtype)
    dc = b.NgcCache(c.k.cuda(), c.v.cuda(), c.seq_off.cuda(), c.lens.cuda(), Hq, t_max)
    out = torch.full((L, B, Hq, t_max, d), 3.0, dtype=torch.float32, device="cuda")
    st = b.new_status()
    if R:
        b.ngc_replay_attn(dc, q.cuda(), out, torch.as_tensor(pos).cuda(), torch.as_tensor(cnt).cuda(),
                          torch.as_tensor(total_before).cuda(), lists=lists, status=st, variant=variant)
    else:
        b.ngc_replay_attn(dc, q.cuda(), out, lists=lists, status=st, variant=variant)
    torch.cuda.synchronize()
    assert status_value(st) == 0
    got = out.cpu().numpy().astype(np.float64)
    kf, vf, qf = synth.as_f64(synth.to_numpy(c.k)), synth.as_f64(synth.to_numpy(c.v)), synth.as_f64(synth.to_numpy(q))
    so = c.seq_off.numpy()
    for bb in range(B):
        Tb = int(T[bb])
        for l in range(L):
            masks = []
            for h in range(Hkv):
                gi = list_of(lists, l, h, Hkv)
                kept = [pos[r, bb, gi, : cnt[r, bb, gi]] for r in range(R)]
                masks.append(replay.dense_mask(Tb, [int(x) for x in total_before[:, bb]], kept))
            ref = replay.replay_attention(qf[l, bb, :, :Tb], kf[l, :, so[bb]: so[bb] + Tb], vf[l, :, so[bb]: so[bb] + Tb], np.stack(masks))
            assert max_rel_err_per_vector(got[l, bb, :, :Tb], ref) <= 2e-2, (l, bb)
        assert np.all(got[:, bb, :, Tb:] == 3.0)                  # rows beyond the sequence are not written


VARIANTS = [None, 1]          # the tcgen05 kernel (default path) and the warp-level MMA kernel it replaced


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("lists,block,R,lo,hi", [(0, 1, 3, 20, 150), (1, 1, 4, 5, 90), (2, 4, 3, 30, 200), (1, 32, 2, 100, 300), (0, 1, 6, 1, 12)])
def test_replay_attn_matches_oracle(lists, block, R, lo, hi, variant):
    run_case(2, 2, 4, 2, lists, block, R, lo, hi, tail=[37, 1], seed=10 * R + lists, variant=variant)


@pytest.mark.parametrize("variant", VARIANTS)
def test_replay_attn_without_rounds_is_causal_attention(variant):
    run_case(1, 2, 12, 2, 0, 1, 0, 0, 0, tail=[200, 65], seed=3, variant=variant)


@pytest.mark.parametrize("variant", VARIANTS)
def test_replay_attn_gqa_shape_of_the_model(variant):
    run_case(1, 1, 12, 2, 1, 32, 2, 256, 256, tail=[100], seed=5, variant=variant)


@pytest.mark.parametrize("Hq,Hkv", [(3, 1), (28, 4), (1, 1), (5, 5)])
def test_replay_attn_odd_and_single_head_groups(Hq, Hkv):
    """The tcgen05 kernel takes the heads of a KV group two at a time: groups of 3 and 7 leave the last pair half
    empty, groups of 1 run one head per CTA."""
    run_case(1, 2, Hq, Hkv, 1, 1, 3, 40, 160, tail=[77, 130], seed=40 + Hq)


def test_replay_attn_running_maximum_moves_many_times():
    """Keys that grow along the sequence: the accumulator in tensor memory has to be rescaled again and again (the
    kernel moves its reference maximum only when the true one has grown by more than a factor 2^8)."""
    run_case(1, 2, 4, 2, 0, 1, 2, 150, 300, tail=[260, 40], seed=9, key_growth=0.05)
    run_case(1, 1, 2, 1, 1, 1, 0, 0, 0, tail=[700], seed=11, key_growth=0.02)


def test_replay_attn_many_rounds_inside_one_query_tile():
    """Rounds every few tokens: a 128-token query tile straddles dozens of eviction rounds, each with its own kept list."""
    run_case(1, 2, 2, 1, 0, 1, 30, 5, 9, tail=[9, 3], seed=13)


def test_replay_attn_more_rounds_in_a_tile_than_the_table_holds_is_reported():
    """A round every other token puts more than 33 eviction rounds inside one 128-token query tile; the tcgen05 kernel
    keeps a fixed table per tile, so it reports the sequence (bad counts) instead of computing a wrong answer silently,
    and returns normally."""
    b = ngc()
    rng = np.random.default_rng(5)
    R, B, G, L, Hq, Hkv, d = 50, 1, 1, 1, 2, 1, 128
    ks, budget, alive_before, total_before = random_history(rng, R, B, G, 1, 2, 2)
    pos, cnt, st0 = gpu_replay(ks, budget, alive_before, total_before, 1, int(alive_before.max()))
    assert st0 == 0
    T = int(total_before[-1, 0]) + 5
    c = synth.make_cache(L, B, Hq, Hkv, d, torch.bfloat16, [T], capacity=T, seed=1)
    dc = b.NgcCache(c.k.cuda(), c.v.cuda(), c.seq_off.cuda(), c.lens.cuda(), Hq, T)
    q = synth.normal((L, B, Hq, T, d), 2, torch.bfloat16).cuda()
    out = torch.zeros((L, B, Hq, T, d), dtype=torch.float32, device="cuda")
    st = b.new_status()
    b.ngc_replay_attn(dc, q, out, torch.as_tensor(pos).cuda(), torch.as_tensor(cnt).cuda(), torch.as_tensor(total_before).cuda(), status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 1
    assert bool(torch.isfinite(out).all())
