"""Seeded random shapes for the decode kernels against the oracle: group sizes 1..16 and beyond,
few and many strips (with and without token splits), empty / one-token / tile-border lengths,
layer ranges, appends, contiguous and paged layouts."""
import numpy as np
import pytest
import torch

import oracle
from helpers import max_rel_err_per_vector, ngc, status_value, to_device_cache
from paper_2604_18002_b200 import synth
from test_gpu_paged import check_logical_equals, to_paged

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", list(range(12)))
def test_decode_random_shapes(seed):
    b = ngc()
    rng = np.random.default_rng(1000 + seed)
    d, dtype = 128, torch.bfloat16
    Hkv = int(rng.choice([1, 2, 4]))
    g = int(rng.choice([1, 2, 3, 6, 7, 8, 12, 16, 20]))
    Hq = Hkv * g
    L = int(rng.integers(1, 4))
    B = int(rng.choice([1, 2, 5, 40]))
    max_len = int(rng.choice([70, 300, 1500, 5000])) if B < 40 else int(rng.choice([70, 300]))
    lens = rng.integers(0, max_len + 1, B).astype(np.int32)
    lens[rng.integers(0, B)] = max_len
    special = [0, 1, 63, 64, 65, 128]
    for i in range(min(B, 3)):
        if rng.random() < 0.5:
            lens[i] = min(max_len, special[rng.integers(0, len(special))])
    steps = 3
    cap = max_len + steps
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=cap, seed=seed, outlier_channels=4)
    dc = to_device_cache(c, cap)
    k_ref, v_ref = synth.to_numpy(c.k).copy(), synth.to_numpy(c.v).copy()
    so, o_lens = c.seq_off.numpy(), lens.copy()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, dc))
    st = b.new_status()
    out = torch.zeros((L, B, Hq, d), dtype=torch.float32, device="cuda")
    for s in range(steps):
        q = synth.make_queries(L, B, Hq, d, dtype, seed=seed * 10 + s)
        nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=seed * 10 + 5 + s)
        if L > 1 and s == 1:        # the same step issued as two calls over layer ranges
            b.ngc_decode_attn_ragged(dc, q.cuda(), out, nk.cuda(), nv.cuda(), layer_begin=0, layer_end=1, ws=ws, status=st)
            b.ngc_decode_attn_ragged(dc, q.cuda(), out, nk.cuda(), nv.cuda(), layer_begin=1, layer_end=L, ws=ws, status=st)
        else:
            b.ngc_decode_attn_ragged(dc, q.cuda(), out, nk.cuda(), nv.cuda(), ws=ws, status=st)
        ref, rc = oracle.decode_attn(k_ref, v_ref, so, o_lens, synth.to_numpy(q), synth.to_numpy(nk), synth.to_numpy(nv))
        assert rc == 0
        assert max_rel_err_per_vector(out.cpu().numpy().astype(np.float64), ref) <= 2e-2, (s, Hq, Hkv, L, B, max_len)
    torch.cuda.synchronize()
    assert status_value(st) == 0 and np.array_equal(dc.lens.cpu().numpy(), o_lens)
    kg, vg = synth.to_numpy(dc.k), synth.to_numpy(dc.v)
    for bb in range(B):
        sl = slice(so[bb], so[bb] + o_lens[bb])
        assert np.array_equal(kg[:, :, sl], k_ref[:, :, sl]) and np.array_equal(vg[:, :, sl], v_ref[:, :, sl])


@pytest.mark.parametrize("seed", list(range(6)))
def test_paged_decode_random_shapes(seed):
    b = ngc()
    rng = np.random.default_rng(2000 + seed)
    d, dtype = 128, torch.bfloat16
    Hkv = int(rng.choice([1, 2, 4]))
    g = int(rng.choice([1, 3, 6, 7, 8, 16]))
    Hq = Hkv * g
    L, B = int(rng.integers(1, 3)), int(rng.choice([1, 3, 30]))
    page = int(rng.choice([32, 64]))
    lists = int(rng.integers(0, 3))
    pages_cap = int(rng.choice([4, 12, 40]))
    cap = pages_cap * page
    steps = 3
    lens = rng.integers(0, cap - steps + 1, B).astype(np.int32)
    lens[0] = cap - steps
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=cap, seed=seed + 50, outlier_channels=4)
    pc = to_paged(c, page, pages_cap, lists, seed=seed)
    k_ref, v_ref = synth.to_numpy(c.k).copy(), synth.to_numpy(c.v).copy()
    so, o_lens = c.seq_off.numpy(), lens.copy()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, pc.as_contiguous_desc()))
    st = b.new_status()
    out = torch.zeros((L, B, Hq, d), dtype=torch.float32, device="cuda")
    for s in range(steps):
        q = synth.make_queries(L, B, Hq, d, dtype, seed=seed * 10 + s)
        nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=seed * 10 + 5 + s)
        b.ngc_decode_attn_paged(pc, q.cuda(), out, nk.cuda(), nv.cuda(), ws=ws, status=st)
        ref, rc = oracle.decode_attn(k_ref, v_ref, so, o_lens, synth.to_numpy(q), synth.to_numpy(nk), synth.to_numpy(nv))
        assert rc == 0
        assert max_rel_err_per_vector(out.cpu().numpy().astype(np.float64), ref) <= 2e-2, (s, Hq, Hkv, L, B, page, lists)
    torch.cuda.synchronize()
    assert status_value(st) == 0 and np.array_equal(pc.lens.cpu().numpy(), o_lens)
    check_logical_equals(pc, k_ref, v_ref, so, o_lens)
