"""Shared helpers of the GPU parity tests: move seeded inputs to the device,
run the CUDA path through the binding, and compare with the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from paper_2604_18002_b200 import synth


def ngc():
    from paper_2604_18002_b200 import binding
    return binding


def to_device_cache(c: synth.Cache, max_len=None):
    b = ngc()
    dev = "cuda"
    if max_len is None:
        max_len = int(c.lens.max()) if c.B else 0
    return b.NgcCache(c.k.to(dev), c.v.to(dev), c.seq_off.to(dev), c.lens.to(dev), c.Hq, max_len)


def status_value(st: torch.Tensor) -> int:
    return int(st.item())


def gpu_sample(logits, n, n_protect, budget, k_max, seed, rnd, greedy=0, list_base=0, want_mask=True):
    b = ngc()
    dev = "cuda"
    lg = torch.as_tensor(np.ascontiguousarray(logits, np.float32)).to(dev)
    B, G, n_max = lg.shape
    n_t = torch.as_tensor(np.asarray(n, np.int32)).to(dev)
    p_t = None if n_protect is None else torch.as_tensor(np.asarray(n_protect, np.int32)).to(dev)
    k_t = torch.as_tensor(np.asarray(budget, np.int32)).to(dev)
    ko = torch.full((B, G, k_max), -7, dtype=torch.int32, device=dev)
    ks = torch.full((B, G, k_max), -7, dtype=torch.int32, device=dev)
    km = torch.full((B, G, n_max), 9, dtype=torch.uint8, device=dev) if want_mask else None
    st = b.new_status()
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_SAMPLE, None, G, n_max, k_max, B=B))
    b.ngc_sample_evict(lg, n_t, p_t, k_t, seed, rnd, ko, ks, km, greedy=greedy, list_base=list_base, ws=ws, status=st)
    torch.cuda.synchronize()
    return ko.cpu().numpy(), ks.cpu().numpy(), (km.cpu().numpy() if want_mask else None), status_value(st)


def gpu_logprob(logits, n, n_protect, budget, kept_order):
    b = ngc()
    dev = "cuda"
    lg = np.ascontiguousarray(logits, np.float32)
    if lg.ndim == 3:
        lg = lg[None]
    NB, B, G, n_max = lg.shape
    ko = np.ascontiguousarray(kept_order, np.int32).reshape(NB, B, G, -1)

    def bc(a):
        return torch.as_tensor(np.ascontiguousarray(np.broadcast_to(np.asarray(a, np.int32).reshape(-1, B), (NB, B)))).to(dev)
    lp = torch.full((NB, B, G), 123.0, dtype=torch.float64, device=dev)
    st = b.new_status()
    b.ngc_evict_logprob(torch.as_tensor(lg).to(dev), bc(n), None if n_protect is None else bc(n_protect), bc(budget),
                        torch.as_tensor(ko).to(dev), lp, status=st)
    torch.cuda.synchronize()
    return lp.cpu().numpy(), status_value(st)


def gpu_logprob_grad(logits, n, n_protect, budget, kept_order, grad_logp=None):
    b = ngc()
    dev = "cuda"
    lg = np.ascontiguousarray(logits, np.float32)
    if lg.ndim == 3:
        lg = lg[None]
    NB, B, G, n_max = lg.shape
    ko = np.ascontiguousarray(kept_order, np.int32).reshape(NB, B, G, -1)

    def bc(a):
        return torch.as_tensor(np.ascontiguousarray(np.broadcast_to(np.asarray(a, np.int32).reshape(-1, B), (NB, B))).copy()).to(dev)
    out = torch.full((NB, B, G, n_max), 77.0, dtype=torch.float32, device=dev)
    up = None if grad_logp is None else torch.as_tensor(np.ascontiguousarray(np.broadcast_to(grad_logp, (NB, B, G)), np.float64).copy()).to(dev)
    st = b.new_status()
    b.ngc_evict_logprob_backward(torch.as_tensor(lg).to(dev), bc(n), None if n_protect is None else bc(n_protect), bc(budget),
                                 torch.as_tensor(ko).to(dev), out, up, status=st)
    torch.cuda.synchronize()
    return out.cpu().numpy(), status_value(st)


def max_rel_err_per_vector(got: np.ndarray, ref: np.ndarray) -> float:
    """max over (.., head) vectors of ||got - ref||_inf / ||ref||_inf."""
    num = np.abs(got.astype(np.float64) - ref).max(-1)
    den = np.abs(ref).max(-1)
    den = np.where(den == 0, 1.0, den)
    return float((num / den).max()) if num.size else 0.0
