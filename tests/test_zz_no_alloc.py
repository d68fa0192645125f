"""The workspace-free decode entry (collected last on purpose).

``ngc_decode_attn_ragged_static`` serves callers that cannot give the library
device scratch memory (no access to the allocator, all memory owned by a host
framework's pool, no tolerance for cudaMalloc's device-wide stall): its split
partials live in an array built into the library image.  It must give the same
result as the workspace entry, call after call, because the shared array keeps
the previous call's contents; both are also held against the CPU oracle, and
the device's free memory must not move across a call.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import max_rel_err_per_vector, ngc, status_value, to_device_cache
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu


def _case(dtype, L, B, Hq, Hkv, d, lens, cap, seed):
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=cap, seed=seed, outlier_channels=4 if d == 128 else 0)
    q = synth.make_queries(L, B, Hq, d, dtype, seed=seed + 1)
    nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=seed + 2)
    return c, q, nk, nv


@pytest.mark.parametrize("dtype,Hq,Hkv,d,tol", [(torch.bfloat16, 12, 2, 128, 2e-2), (torch.float32, 4, 4, 64, 1e-5)])
def test_static_scratch_decode_matches_workspace_decode_twice(dtype, Hq, Hkv, d, tol):
    b = ngc()
    L, B = 2, 2
    # few strips, long sequences: the launch splits along tokens, so the scratch is really used
    results = []
    for call, (lens, seed) in enumerate([([3000, 1100], 5), ([2500, 40], 9)]):
        c, q, nk, nv = _case(dtype, L, B, Hq, Hkv, d, lens, 3001, seed)
        ref_cache = to_device_cache(c, 3001)
        assert b.decode_splits(ref_cache) > 1
        ws = b.alloc_workspace(b.workspace_bytes(b.OP_DECODE, ref_cache))
        ref = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
        st = b.new_status()
        b.ngc_decode_attn_ragged(ref_cache, q.cuda(), ref, nk.cuda(), nv.cuda(), ws=ws, status=st)
        got_cache = to_device_cache(c, 3001)
        got = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
        qd, nkd, nvd = q.cuda(), nk.cuda(), nv.cuda()
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        b.ngc_decode_attn_ragged_static(got_cache, qd, got, nkd, nvd, status=st)
        torch.cuda.synchronize()
        if call > 0:      # (the first call of a process may load the kernels' code; from then on nothing may move)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert status_value(st) == 0
        # the oracle on the same bytes (its cache copy takes the appended row itself)
        ok, ov, ol = synth.to_numpy(c.k).copy(), synth.to_numpy(c.v).copy(), c.lens.numpy().copy()
        want, rc = oracle.decode_attn(ok, ov, c.seq_off.numpy(), ol, synth.to_numpy(q), synth.to_numpy(nk), synth.to_numpy(nv))
        assert rc == 0
        if dtype == torch.float32:
            assert np.max(np.abs(got.cpu().numpy() - want)) <= tol
        else:
            assert max_rel_err_per_vector(got.cpu().numpy(), want) <= tol
        assert np.array_equal(got_cache.lens.cpu().numpy(), ol)
        r, g = ref.cpu().numpy().astype(np.float64), got.cpu().numpy()
        assert np.isfinite(g).all()
        if dtype == torch.float32:
            assert np.max(np.abs(g - r)) <= tol
        else:
            assert max_rel_err_per_vector(g, r) <= tol
        assert torch.equal(got_cache.lens, ref_cache.lens)
        assert torch.equal(got_cache.k, ref_cache.k) and torch.equal(got_cache.v, ref_cache.v)
        results.append(g)
    assert not np.array_equal(results[0], results[1])


def test_static_scratch_refuses_oversized_launch():
    b = ngc()
    # one layer, 64 long sequences of a 28-head model: the partials would not fit the built-in array
    L, B, Hq, Hkv, d = 1, 8, 64, 1, 128
    k = torch.zeros((L, Hkv, B * 20000, d), dtype=torch.bfloat16, device="cuda")
    cache = b.NgcCache(k, k.clone(), torch.arange(0, B + 1, dtype=torch.int64, device="cuda") * 20000,
                       torch.full((B,), 19000, dtype=torch.int32, device="cuda"), Hq, 20000)
    need = b.workspace_bytes(b.OP_DECODE, cache)
    assert need > b.STATIC_SCRATCH_BYTES
    q = torch.zeros((L, B, Hq, d), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((L, B, Hq, d), dtype=torch.float32, device="cuda")
    with pytest.raises(b.NgcError, match="NGC_STATIC_SCRATCH_BYTES"):
        b.ngc_decode_attn_ragged_static(cache, q, out)


def test_static_scratch_refuses_a_stream_of_another_device():
    """The built-in array exists once per GPU; the entry uses the current device's copy and must refuse a stream
    that belongs to another device instead of enqueueing kernels that would write through a foreign address."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two CUDA devices")
    b = ngc()
    c, q, nk, nv = _case(torch.bfloat16, 1, 1, 12, 2, 128, [300], 301, 3)
    cache = to_device_cache(c, 301)
    out = torch.zeros(q.shape, dtype=torch.float32, device="cuda")
    other = torch.cuda.Stream(device=1)
    with pytest.raises(b.NgcError):
        with torch.cuda.stream(other):
            torch.cuda.set_device(0)          # stream of device 1, device 0 current
            b.ngc_decode_attn_ragged_static(cache, q.cuda(0), out)
    torch.cuda.set_device(0)
