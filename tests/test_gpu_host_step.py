"""The host-buffer entry (pinned inputs in, results out, copies overlapped with compute) must give
exactly what the device-resident call sequence gives, with and without the double-buffered cache
upload that is pipelined across steps; one step is also checked against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import max_rel_err_per_vector, ngc
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu


def make_step_inputs(i, L, B, Hq, Hkv, d, T, steps, dtype):
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, [T] * B, capacity=T, seed=100 + i, outlier_channels=4)
    pin = lambda t: t.contiguous().pin_memory()
    return dict(k=pin(c.k), v=pin(c.v), lens=pin(c.lens), logits=pin(synth.make_logits(B, 1, T, seed=200 + i)),
                q=pin(synth.make_queries(L, B, Hq, d, dtype, seed=300 + i, steps=steps)),
                nk=pin(synth.make_new_kv(L, B, Hkv, d, dtype, seed=400 + 2 * i, steps=steps)[0]),
                nv=pin(synth.make_new_kv(L, B, Hkv, d, dtype, seed=400 + 2 * i, steps=steps)[1]),
                qr=pin(synth.normal((L, B, Hq, 5, d), 500 + i, dtype)), so=c.seq_off)


@pytest.mark.parametrize("double_buffer", [False, True])
def test_host_step_equals_device_resident_sequence(double_buffer):
    b = ngc()
    from paper_2604_18002_b200.rollout import HostStep, NgcRollout
    L, B, Hq, Hkv, d, T, K, steps, dtype = 2, 3, 12, 2, 128, 320, 150, 5, torch.bfloat16
    n_steps = 3
    inputs = [make_step_inputs(i, L, B, Hq, Hkv, d, T, steps, dtype) for i in range(n_steps)]
    n_t = torch.full((B,), T, dtype=torch.int32, device="cuda")
    k_t = torch.full((B,), K, dtype=torch.int32, device="cuda")

    def fresh():
        return NgcRollout(L, B, Hq, Hkv, d, dtype, capacity=T, n_max=T, k_max=K, device="cuda")

    # device-resident reference: same calls, inputs copied by hand
    want = []
    ro = fresh()
    for i, x in enumerate(inputs):
        ro.cache.k.copy_(x["k"]); ro.cache.v.copy_(x["v"]); ro.cache.lens.copy_(x["lens"])
        lg = x["logits"].cuda()
        ro.eviction_round(n_t, None, k_t, 9, i, q_recent=x["qr"].cuda(), logits=lg)
        outs = torch.empty((steps, L, B, Hq, d), dtype=torch.float32, device="cuda")
        for s in range(steps):
            ro.decode_step(x["q"][s].cuda(), outs[s], x["nk"][s].cuda(), x["nv"][s].cuda())
        torch.cuda.synchronize()
        ro.check_status()
        want.append((ro.kept_order.cpu().clone(), ro.logp.cpu().clone(), outs.cpu().clone()))

    ro = fresh()
    hs = HostStep(ro, steps, chunk=2, double_buffer=double_buffer)
    d_qr = torch.empty((L, B, Hq, 5, d), dtype=dtype, device="cuda")
    for i, x in enumerate(inputs):
        h_out = torch.empty((steps, L, B, Hq, d), dtype=torch.float32).pin_memory()
        h_ko = torch.empty(ro.kept_order.shape, dtype=torch.int32).pin_memory()
        h_lp = torch.empty(ro.logp.shape, dtype=torch.float64).pin_memory()
        nxt = inputs[i + 1] if i + 1 < n_steps else None
        h2d, d2h = hs.run(x["k"], x["v"], x["lens"], x["logits"], x["q"], x["nk"], x["nv"], h_out, h_ko, h_lp, n_t, None, k_t, 9, i,
                          h_q_recent=x["qr"], d_q_recent=d_qr, prefetch_next=(nxt["k"], nxt["v"]) if nxt else None)
        torch.cuda.synchronize()
        ro.check_status()
        assert torch.equal(h_ko, want[i][0]) and torch.equal(h_lp, want[i][1]) and torch.equal(h_out, want[i][2])
        assert d2h == h_out.numel() * 4 + h_ko.numel() * 4 + h_lp.numel() * 8 and h2d > x["q"].numel() * 2
    # the last step against the oracle
    x = inputs[-1]
    lens = np.full(B, T, np.int32)
    budget = np.full(B, K, np.int32)
    r_ko, r_ks, _, _ = oracle.sample_evict(x["logits"].numpy(), lens, None, budget, K, seed=9, rnd=n_steps - 1)
    assert np.array_equal(want[-1][0].numpy(), r_ko)
    kc, vc, nl, rc = oracle.compact_kv(synth.to_numpy(x["k"]), synth.to_numpy(x["v"]), x["so"].numpy(), lens, r_ks, budget, 0)
    ol = nl.copy()
    for s in range(steps):
        ref, rc = oracle.decode_attn(kc, vc, x["so"].numpy(), ol, synth.to_numpy(x["q"][s]), synth.to_numpy(x["nk"][s]), synth.to_numpy(x["nv"][s]))
        assert rc == 0 and max_rel_err_per_vector(want[-1][2][s].numpy().astype(np.float64), ref) <= 2e-2
