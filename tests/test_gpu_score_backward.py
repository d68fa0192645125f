"""ngc_score_evict_backward against the CPU oracle (chain rule through block mean, row average and
softmax, in double).  bf16 cache, bf16 MMA operands (dz is rounded to bf16) and a bf16 grad_k: the
bar is 2e-2 of the largest entry of each gradient tensor, per sequence, plus 1e-6 absolute (a
sequence whose tokens all fall into one unit has a gradient that cancels exactly in exact arithmetic;
what the kernel leaves there is rounding noise of terms of size |grad_logits| / sqrt(d))."""
import numpy as np
import pytest
import torch

import oracle
from helpers import ngc, status_value, to_device_cache
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 2e-2
FLOOR = 1e-6


def run_case(L, B, Hq, Hkv, w, lens, lists, block, log_transform, seed):
    b = ngc()
    d, dtype = 128, torch.bfloat16
    cap = max(lens) + 5
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=cap, seed=seed, outlier_channels=4)
    qr = synth.normal((L, B, Hq, w, d), seed + 1, dtype)
    G = oracle.lists_G(lists, L, Hkv)
    n_max = (cap + block - 1) // block
    up = synth.make_logits(B, G, n_max, seed=seed + 2).numpy().astype(np.float64)
    k_np, so, ln = synth.to_numpy(c.k), c.seq_off.numpy(), c.lens.numpy()
    ref_q, ref_k = oracle.score_evict_grad(k_np, so, ln, synth.to_numpy(qr), block, lists, up, log_transform=log_transform)
    dc = to_device_cache(c, cap)
    st = b.new_status()
    logits = torch.full((B, G, n_max), 0.0, dtype=torch.float32, device="cuda")
    ws_f = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE, dc, G, n_max))
    b.ngc_score_evict(dc, qr.cuda(), block, lists, logits, log_transform=log_transform, ws=ws_f, status=st)
    gq = torch.full(qr.shape, 9.0, dtype=torch.float32, device="cuda")
    gk = torch.zeros_like(dc.k)
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE_BACKWARD, dc))
    b.ngc_score_evict_backward(dc, qr.cuda(), block, lists, torch.as_tensor(up, dtype=torch.float32).cuda(), gq, gk,
                               logits=logits, log_transform=log_transform, ws=ws, status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 0
    got_q = gq.cpu().numpy().astype(np.float64)
    got_k = synth.as_f64(synth.to_numpy(gk))
    for bb in range(B):
        sl = slice(so[bb], so[bb] + ln[bb])
        sq = np.abs(ref_q[:, bb]).max()
        sk = np.abs(ref_k[:, :, sl]).max() if ln[bb] else 0.0
        assert np.max(np.abs(got_q[:, bb] - ref_q[:, bb])) <= TOL * sq + FLOOR, ("dq", bb)
        if ln[bb]:
            assert np.max(np.abs(got_k[:, :, sl] - ref_k[:, :, sl])) <= TOL * sk + FLOOR, ("dk", bb)
        dead = slice(so[bb] + ln[bb], so[bb + 1])
        assert np.all(got_k[:, :, dead] == 0.0)            # rows beyond the sequence are not written
    return got_q, got_k


@pytest.mark.parametrize("Hq,Hkv,w,lists,block,log_transform", [
    (12, 2, 5, 1, 1, 0), (12, 2, 5, 0, 32, 0), (28, 4, 5, 2, 1, 0), (12, 2, 5, 1, 32, 1), (8, 2, 3, 2, 5, 1), (4, 4, 1, 1, 1, 0)])
def test_score_backward_matches_oracle(Hq, Hkv, w, lists, block, log_transform):
    run_case(2, 4, Hq, Hkv, w, [3, 64, 257, 900], lists, block, log_transform, seed=31 + Hq + w)


def test_score_backward_token_ranges_and_unsupported_shapes():
    b = ngc()
    run_case(1, 1, 12, 2, 5, [3000], 1, 1, 0, seed=5)      # one long strip: several token ranges per strip
    c = synth.make_cache(1, 1, 4, 4, 64, torch.float32, [10], capacity=10, seed=1)
    dc = to_device_cache(c, 10)
    qr = synth.normal((1, 1, 4, 2, 64), 2, torch.float32).cuda()
    with pytest.raises(b.NgcError, match="not supported"):
        b.ngc_score_evict_backward(dc, qr, 1, 1, torch.zeros((1, 1, 10), device="cuda"), torch.zeros_like(qr), torch.zeros_like(dc.k))


@pytest.mark.parametrize("Hq,Hkv,w,lens", [
    (16, 2, 5, [127, 128, 129, 255, 256, 257, 1, 4]),      # 40 rows, the widest strip; lengths around the 128-token tiles;
                                                           # fewer tokens than window queries
    (4, 2, 16, [15, 16, 17, 384]),                         # exactly 32 rows with the longest window
    (12, 2, 5, [0, 2, 640]),                               # an empty sequence beside live ones
])
def test_score_backward_tile_edges_and_row_counts(Hq, Hkv, w, lens):
    run_case(2, len(lens), Hq, Hkv, w, lens, 1, 1, 0, seed=3 * Hq + w)
    run_case(1, len(lens), Hq, Hkv, w, lens, 2, 8, 1, seed=5 * Hq + w)


def test_score_backward_cache_smaller_than_one_tile():
    """A whole cache plane shorter than one 128-token tile (the tensor-map boxes reach beyond the tensor)."""
    run_case(1, 1, 4, 2, 2, [10], 1, 1, 0, seed=2)
    run_case(2, 2, 12, 2, 5, [1, 7], 2, 4, 1, seed=3)


def test_score_backward_many_short_strips_write_grad_q_directly():
    """More strips than the kernels want items: no strip is cut into token ranges and the gradient pass writes
    grad_q itself (no partials, no reduction launch)."""
    rng = np.random.default_rng(7)
    lens = [int(x) for x in rng.integers(0, 300, size=80)]
    lens[3] = 0
    lens[5] = 128
    run_case(4, 80, 4, 2, 3, lens, 1, 32, 0, seed=11)


def test_score_backward_with_a_length_per_layer():
    """Per-layer lists whose layers hold different numbers of tokens: every layer against the oracle run on it alone."""
    b = ngc()
    L, B, Hq, Hkv, d, w, block, dtype = 3, 2, 12, 2, 128, 5, 32, torch.bfloat16
    cap = 400
    lens = np.array([[300, 268, 290], [65, 97, 33]], np.int32)               # [B][L]
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, [cap, cap], capacity=cap, seed=3, outlier_channels=4)
    qr = synth.normal((L, B, Hq, w, d), 4, dtype)
    n_max = (cap + block - 1) // block
    up = synth.make_logits(B, L, n_max, seed=5).numpy().astype(np.float64)
    dc = b.NgcCache(c.k.cuda(), c.v.cuda(), c.seq_off.cuda(), torch.as_tensor(lens).cuda(), Hq, cap, b.LISTS_PER_LAYER)
    gq = torch.zeros(qr.shape, dtype=torch.float32, device="cuda")
    gk = torch.zeros_like(dc.k)
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE_BACKWARD, dc))
    st = b.new_status()
    b.ngc_score_evict_backward(dc, qr.cuda(), block, b.LISTS_PER_LAYER, torch.as_tensor(up, dtype=torch.float32).cuda(), gq, gk, ws=ws, status=st)
    torch.cuda.synchronize()
    assert status_value(st) == 0
    so = c.seq_off.numpy()
    for l in range(L):
        ref_q, ref_k = oracle.score_evict_grad(np.ascontiguousarray(synth.to_numpy(c.k)[l:l + 1]), so, np.ascontiguousarray(lens[:, l]),
                                               np.ascontiguousarray(synth.to_numpy(qr)[l:l + 1]), block, 0, np.ascontiguousarray(up[:, l:l + 1]))
        got_q = gq[l:l + 1].cpu().numpy().astype(np.float64)
        got_k = synth.as_f64(synth.to_numpy(gk[l:l + 1]))
        for bb in range(B):
            sl = slice(so[bb], so[bb] + lens[bb, l])
            assert np.max(np.abs(got_q[:, bb] - ref_q[:, bb])) <= TOL * np.abs(ref_q[:, bb]).max() + FLOOR
            assert np.max(np.abs(got_k[:, :, sl] - ref_k[:, :, sl])) <= TOL * np.abs(ref_k[:, :, sl]).max() + FLOOR
            assert np.all(got_k[:, :, so[bb] + lens[bb, l]:so[bb + 1]] == 0.0)
