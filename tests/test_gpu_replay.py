"""ngc_replay_visibility against the CPU oracle of Appendix A.3: integer lists, bit-exact.  Small
random multi-round histories (uneven blocks, units of several tokens with a short last unit,
failing lists), the paper's replay-mask figure, and a full-size history shaped like the rollout
loop (64 sequences x 28 per-layer lists x 16 rounds, 768 -> 256)."""
import json
import os

import numpy as np
import pytest
import torch

from helpers import ngc, status_value
from oracle import replay

pytestmark = pytest.mark.gpu


def gpu_replay(ks, budget, alive_before, total_before, block, alive_max):
    b = ngc()
    R, B, G, k_max = ks.shape
    t = lambda a: torch.as_tensor(np.ascontiguousarray(a, np.int32)).cuda()
    pos = torch.full((R, B, G, k_max * block), -9, dtype=torch.int32, device="cuda")
    cnt = torch.full((R, B, G), -9, dtype=torch.int32, device="cuda")
    st = b.new_status()
    b.ngc_replay_visibility(t(ks), t(budget), t(alive_before), t(total_before), block, alive_max, pos, cnt, status=st)
    torch.cuda.synchronize()
    return pos.cpu().numpy(), cnt.cpu().numpy(), status_value(st)


def random_history(rng, R, B, G, block, grow_lo, grow_hi):
    grows = rng.integers(grow_lo, grow_hi + 1, (R, B))
    alive_before = np.zeros((R, B), np.int32)
    total_before = np.cumsum(grows, 0).astype(np.int32)
    budget = np.zeros((R, B), np.int32)
    kept_n = np.zeros(B, np.int64)
    per_round = []
    for r in range(R):
        alive_before[r] = kept_n + grows[r]
        n_units = (alive_before[r] + block - 1) // block
        budget[r] = [rng.integers(0, n + 1) for n in n_units]
        per_round.append(n_units)
        # all lists of a sequence keep the same unit count; token counts may differ by the short unit,
        # so the next round's alive count is only defined when the last unit is full or never short
        kept_n = budget[r].astype(np.int64) * block
        alive_fix = alive_before[r] % block
        kept_n = np.where((alive_fix != 0) & (budget[r] == n_units), kept_n - (block - alive_fix), kept_n)
    k_max = max(1, int(budget.max()))
    ks = np.full((R, B, G, k_max), -1, np.int32)
    for r in range(R):
        for b in range(B):
            for g in range(G):
                n_units = int(per_round[r][b])
                K = int(budget[r, b])
                if K == n_units:
                    units = np.arange(n_units)
                else:     # never keep the (possibly short) last unit unless everything is kept: equal token counts
                    units = np.sort(rng.choice(max(n_units - 1, 1), K, replace=False)) if K else np.zeros(0, int)
                ks[r, b, g, :K] = units
    return ks, budget, alive_before, total_before


@pytest.mark.parametrize("R,B,G,block,lo,hi", [(4, 3, 2, 1, 2, 40), (5, 2, 3, 4, 5, 70), (3, 4, 1, 32, 40, 300), (1, 2, 2, 1, 1, 5)])
def test_replay_visibility_matches_oracle(R, B, G, block, lo, hi):
    rng = np.random.default_rng(R * 100 + block)
    ks, budget, alive_before, total_before = random_history(rng, R, B, G, block, lo, hi)
    # the history generator keeps full units unless all are kept; fix the rounds where a short last unit made counts differ
    ref_pos, ref_cnt, rc = replay.alive_positions(ks, budget, alive_before, total_before, block)
    got_pos, got_cnt, st = gpu_replay(ks, budget, alive_before, total_before, block, int(alive_before.max()))
    assert st == rc
    assert np.array_equal(got_cnt, ref_cnt) and np.array_equal(got_pos, ref_pos)


def test_replay_visibility_figure_and_failures():
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "replay_mask_figure.json")))
    ks = np.array([[[[0, 2, 4, -1]]], [[[0, 2, 4, 5]]]], np.int32)          # round 1 evicts t1, t3; round 2 evicts t2, t5
    pos, cnt, st = gpu_replay(ks, [[3], [4]], [[5], [6]], [[5], [8]], 1, 6)
    assert st == 0 and list(cnt.ravel()) == [3, 4]
    assert list(pos[0, 0, 0, :3]) == [0, 2, 4] and list(pos[1, 0, 0]) == g["final_survivors"]
    M = replay.dense_mask(g["tokens"], [5, 8], [pos[0, 0, 0, :3], pos[1, 0, 0]])
    for row, vis in g["visible"].items():
        assert list(np.nonzero(M[int(row)])[0]) == vis
    # a corrupt list fails from its round on, the other list of the call is unaffected
    ks2 = np.repeat(ks, 2, axis=2)
    ks2[1, 0, 1] = [0, 2, 2, 5]
    pos, cnt, st = gpu_replay(ks2, [[3], [4]], [[5], [6]], [[5], [8]], 1, 6)
    ref_pos, ref_cnt, rc = replay.alive_positions(ks2, [[3], [4]], [[5], [6]], [[5], [8]], 1)
    assert st == 3 and rc == 3 and np.array_equal(cnt, ref_cnt) and np.array_equal(pos, ref_pos)
    pos, cnt, st = gpu_replay(ks, [[3], [4]], [[5], [2]], [[5], [8]], 1, 6)   # fewer alive than the last round kept
    assert st == 1 and list(cnt.ravel()) == [3, -1]


def test_replay_visibility_rollout_loop_size():
    """16 rounds, 64 sequences, 28 per-layer lists, 768 alive -> 256 kept, 512 new tokens per round."""
    rng = np.random.default_rng(11)
    R, B, G, K, peak, delta = 16, 64, 28, 256, 768, 512
    u = rng.random((R, B, G, peak))
    ks = np.sort(np.argsort(u, -1)[..., :K], -1).astype(np.int32)
    budget = np.full((R, B), K, np.int32)
    alive_before = np.full((R, B), peak, np.int32)
    total_before = (peak + delta * np.arange(R))[:, None].repeat(B, 1).astype(np.int32)
    got_pos, got_cnt, st = gpu_replay(ks, budget, alive_before, total_before, 1, peak)
    assert st == 0 and np.all(got_cnt == K)
    sel = [0, 17, 63]
    ref_pos, ref_cnt, rc = replay.alive_positions(ks[:, sel], budget[:, sel], alive_before[:, sel], total_before[:, sel], 1)
    assert rc == 0 and np.array_equal(got_pos[:, sel], ref_pos)
    # properties that hold for every list: ascending, inside the sequence, survivors of round r-1 or new tokens
    assert np.all(np.diff(got_pos, axis=-1) > 0)
    assert np.all(got_pos[-1] < total_before[-1][:, None, None])
    for r in range(1, R):
        old = got_pos[r] < total_before[r - 1][:, None, None]
        assert np.all(old.sum(-1) == (ks[r] < K).sum(-1))


def test_replay_visibility_with_a_length_per_list():
    """Units of 32 tokens, per-layer lists, rounds at lengths that are no multiple of 32: the layers of a sequence
    hold different numbers of tokens, so the alive count is given per (round, sequence, list)."""
    rng = np.random.default_rng(9)
    R, B, G, block = 4, 3, 5, 32
    grows = rng.integers(40, 200, (R, B))
    total_before = np.cumsum(grows, 0).astype(np.int32)
    alive_before = np.zeros((R, B, G), np.int32)
    kept_n = np.zeros((B, G), np.int64)
    budget = np.zeros((R, B), np.int32)
    lists = []
    for r in range(R):
        alive_before[r] = kept_n + grows[r][:, None]
        units = (alive_before[r] + block - 1) // block                      # [B][G]
        budget[r] = np.maximum(1, units.min(1) // 2)
        row = []
        for b in range(B):
            per_g = []
            for g in range(G):
                u = np.sort(rng.choice(units[b, g], budget[r, b], replace=False))
                per_g.append(u)
                short = units[b, g] * block - alive_before[r, b, g]
                kept_n[b, g] = budget[r, b] * block - (short if u[-1] == units[b, g] - 1 else 0)
            row.append(per_g)
        lists.append(row)
    k_max = int(budget.max())
    ks = np.full((R, B, G, k_max), -1, np.int32)
    for r in range(R):
        for b in range(B):
            for g in range(G):
                ks[r, b, g, : budget[r, b]] = lists[r][b][g]
    assert (alive_before.max(2) != alive_before.min(2)).any()              # the lists really differ
    ref_pos, ref_cnt, rc = replay.alive_positions(ks, budget, alive_before, total_before, block)
    got_pos, got_cnt, st = gpu_replay(ks, budget, alive_before, total_before, block, int(alive_before.max()))
    assert rc == 0 and st == 0 and np.array_equal(got_cnt, ref_cnt) and np.array_equal(got_pos, ref_pos)
