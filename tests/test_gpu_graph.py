"""The decode loop replayed as one CUDA graph gives bit-identical results to the eagerly launched loop
(same kernels, same order), for the fp32 tiny shape and a bf16 GQA shape."""
import numpy as np
import pytest
import torch

from helpers import ngc
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,Hq,Hkv,d,T", [(torch.float32, 4, 4, 64, 256), (torch.bfloat16, 12, 2, 128, 300)])
def test_graph_replay_equals_eager_decode_loop(dtype, Hq, Hkv, d, T):
    from paper_2604_18002_b200.rollout import NgcRollout
    L, B, steps = 2, 4, 16
    src = synth.make_cache(L, B, Hq, Hkv, d, dtype, [T, T - 7, 1, 64], capacity=T + 2 * steps + 1, seed=2)
    q = synth.make_queries(L, B, Hq, d, dtype, seed=3, steps=steps).cuda()
    nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=4, steps=steps)
    nk, nv = nk.cuda(), nv.cuda()

    def fresh():
        ro = NgcRollout(L, B, Hq, Hkv, d, dtype, capacity=T + 2 * steps + 1, n_max=8, k_max=8, device="cuda", with_score=False)
        ro.cache.k.copy_(src.k); ro.cache.v.copy_(src.v); ro.cache.lens.copy_(src.lens)
        return ro

    eager = fresh()
    out_e = torch.zeros((steps, L, B, Hq, d), dtype=torch.float32, device="cuda")
    for s in range(steps):
        eager.decode_step(q[s], out_e[s], nk[s], nv[s])
    torch.cuda.synchronize()

    ro = fresh()
    warm = torch.zeros((L, B, Hq, d), dtype=torch.float32, device="cuda")
    ro.decode_step(q[0], warm, nk[0], nv[0])                    # configures the kernels outside the capture
    ro.cache.k.copy_(src.k); ro.cache.v.copy_(src.v); ro.cache.lens.copy_(src.lens)
    out_g = torch.zeros_like(out_e)
    torch.cuda.synchronize()
    graph = ro.capture_decode_steps(q, out_g, nk, nv)
    ro.cache.k.copy_(src.k); ro.cache.v.copy_(src.v); ro.cache.lens.copy_(src.lens)   # capture does not execute
    out_g.zero_()
    graph.replay()
    torch.cuda.synchronize()
    ro.check_status()
    assert torch.equal(out_g, out_e)
    assert torch.equal(ro.cache.lens, eager.cache.lens) and torch.equal(ro.cache.k, eager.cache.k)
    # a second replay continues the rollout from the current lengths
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(ro.cache.lens, eager.cache.lens + steps)
