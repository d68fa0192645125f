"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds NONE of the method's arithmetic: it only draws tensors with a
seeded ``torch.Generator`` and lays them out the way the library expects.  Both
the CUDA path and the CPU oracle receive the very same bytes (the oracle through
:func:`to_numpy`).  The stream depends on (seed, device type): data generated
on the GPU for the large benchmark shapes is copied back to the host for the
oracle, never regenerated.

Cache layout: ``k``/``v`` are ``[L][Hkv][R][d]`` with ``R = seq_off[B]`` rows per
(layer, KV head) plane; sequence ``b`` owns rows ``seq_off[b] .. seq_off[b+1]``
of every plane, of which the first ``lens[b]`` are alive.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch


@dataclass
class Cache:
    k: torch.Tensor        # [L][Hkv][R][d]
    v: torch.Tensor
    seq_off: torch.Tensor  # int64 [B+1]
    lens: torch.Tensor     # int32 [B]
    L: int
    B: int
    Hq: int
    Hkv: int
    d: int

    @property
    def rows(self) -> int:
        return int(self.k.shape[2])

    def clone(self) -> "Cache":
        return Cache(self.k.clone(), self.v.clone(), self.seq_off.clone(), self.lens.clone(),
                     self.L, self.B, self.Hq, self.Hkv, self.d)

    def to(self, device) -> "Cache":
        return Cache(self.k.to(device), self.v.to(device), self.seq_off.to(device), self.lens.to(device),
                     self.L, self.B, self.Hq, self.Hkv, self.d)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal(shape, seed: int, dtype=torch.float32, std: float = 1.0, device="cpu") -> torch.Tensor:
    """N(0, std^2) tensor drawn in fp32 and rounded once to ``dtype``."""
    t = torch.randn(shape, generator=_gen(seed, device), dtype=torch.float32, device=device)
    if std != 1.0:
        t.mul_(std)
    return t.to(dtype)


def make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=None, seed=0, outlier_channels=0,
               outlier_scale=8.0, device="cpu", fill_dead_rows=True, layers=None) -> Cache:
    """K, V ~ N(0,1); optionally ``outlier_channels`` channels of K per (layer, KV head),
    fixed over tokens, scaled by ``outlier_scale`` (the channels are the first entries of a
    seeded permutation of 0..d-1).  ``capacity`` (scalar or per-sequence) is the row capacity
    of each sequence; rows at or beyond ``lens[b]`` hold random data too unless
    ``fill_dead_rows`` is False (then zeros).  Every (layer, KV head) plane has a seed of its own,
    so ``layers`` (a list of layer indices) draws just those layers of the L-layer cache, with the
    same bytes they have in the full one: ``k``/``v`` are then ``[len(layers)][Hkv][R][d]``."""
    lens = torch.as_tensor(lens, dtype=torch.int32).reshape(B)
    if capacity is None:
        cap = lens.to(torch.int64)
    else:
        cap = torch.as_tensor(capacity, dtype=torch.int64).expand(B).clone()
    assert bool((cap >= lens).all())
    seq_off = torch.zeros(B + 1, dtype=torch.int64)
    seq_off[1:] = torch.cumsum(cap, 0)
    R = int(seq_off[-1])
    layer_ids = list(range(L)) if layers is None else [int(l) for l in layers]
    k = torch.empty((len(layer_ids), Hkv, R, d), dtype=dtype, device=device)
    v = torch.empty((len(layer_ids), Hkv, R, d), dtype=dtype, device=device)
    # plane by plane keeps the fp32 staging buffer small for the large shapes
    for li, l in enumerate(layer_ids):
        for h in range(Hkv):
            kp = torch.randn((R, d), generator=_gen(seed * 1000003 + (l * Hkv + h) * 2 + 11, device),
                             dtype=torch.float32, device=device)
            if outlier_channels:
                perm = torch.randperm(d, generator=_gen(seed * 7919 + l * Hkv + h + 5, "cpu"))[:outlier_channels]
                kp[:, perm.to(device)] *= outlier_scale
            k[li, h] = kp.to(dtype)
            vp = torch.randn((R, d), generator=_gen(seed * 1000003 + (l * Hkv + h) * 2 + 12, device),
                             dtype=torch.float32, device=device)
            v[li, h] = vp.to(dtype)
    if not fill_dead_rows:
        for b in range(B):
            k[:, :, int(seq_off[b]) + int(lens[b]):int(seq_off[b + 1])] = 0
            v[:, :, int(seq_off[b]) + int(lens[b]):int(seq_off[b + 1])] = 0
    return Cache(k, v, seq_off.to(device), lens.to(device), len(layer_ids), B, Hq, Hkv, d)


def make_logits(B, G, n_max, seed, std=1.0, device="cpu") -> torch.Tensor:
    return normal((B, G, n_max), seed, torch.float32, std, device)


def make_queries(L, B, Hq, d, dtype, seed, steps=None, device="cpu") -> torch.Tensor:
    shape = (L, B, Hq, d) if steps is None else (steps, L, B, Hq, d)
    return normal(shape, seed, dtype, 1.0, device)


def make_new_kv(L, B, Hkv, d, dtype, seed, steps=None, device="cpu"):
    shape = (L, B, Hkv, d) if steps is None else (steps, L, B, Hkv, d)
    return normal(shape, seed, dtype, 1.0, device), normal(shape, seed + 1, dtype, 1.0, device)


def ragged_lens(B, lo, hi, seed) -> torch.Tensor:
    """Cache lengths uniform in [lo, hi]."""
    r = torch.randint(lo, hi + 1, (B,), generator=_gen(seed, "cpu"), dtype=torch.int64)
    return r.to(torch.int32)


def to_numpy(t: torch.Tensor) -> np.ndarray:
    """Host numpy view of a tensor; bfloat16 becomes its uint16 bit pattern."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 values (exact)."""
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def as_f64(a: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f64(a) if a.dtype == np.uint16 else a.astype(np.float64)


# ---- the five benchmark / parity workloads ----------------------------------

CONFIGS = {
    # name: attention shape, batch, cache, eviction and decode recipe
    1: dict(name="tiny-fp32", L=1, Hq=4, Hkv=4, d=64, dtype="f32", B=4, T=512, n_protect=64, budget=256,
            lists=0, logit_std=1.0, steps=64, outliers=0, data_seed=0, noise_seed=1),
    2: dict(name="1.5B-GQA-B64", L=28, Hq=12, Hkv=2, d=128, dtype="bf16", B=64, T=4096, n_protect=0, budget=2048,
            lists=0, logit_std=math.sqrt(2.0), steps=256, outliers=4, data_seed=0, noise_seed=1),
    3: dict(name="7B-ragged-B256", L=28, Hq=28, Hkv=4, d=128, dtype="bf16", B=256, T=(1024, 8192), n_protect=0,
            budget="third", lists=0, logit_std=1.0, steps=128, outliers=0, data_seed=0, noise_seed=1, len_seed=2),
    4: dict(name="per-head-B128", L=28, Hq=12, Hkv=2, d=128, dtype="bf16", B=128, T=16384, n_protect=0,
            budget=8192, lists=2, logit_std=1.0, steps=64, outliers=0, data_seed=0, noise_seed=1),
    5: dict(name="rollout-loop-B64", L=28, Hq=12, Hkv=2, d=128, dtype="bf16", B=64, T=256, n_protect=0,
            budget=256, lists=1, logit_std=1.0, steps=8192, cadence=512, outliers=0, data_seed=0, noise_seed=1),
    # the paper's own eviction setting: units of 32 tokens, 5 recent queries, one list per layer scored from the
    # real K, half of the units kept each round; 512 = 32 prompts x 16 rollouts, 2048 = 256 prompts x 8 rollouts
    6: dict(name="paper-countdown-B512", L=28, Hq=12, Hkv=2, d=128, dtype="bf16", B=512, T=256, n_protect=0,
            budget=8, block=32, lists=1, logit_std=1.0, steps=1024, cadence=256, outliers=0, data_seed=0, noise_seed=1),
    7: dict(name="paper-math-B2048", L=28, Hq=12, Hkv=2, d=128, dtype="bf16", B=2048, T=352, n_protect=0,
            budget=11, block=32, lists=1, logit_std=1.0, steps=1056, cadence=352, outliers=0, data_seed=0, noise_seed=1),
    # the same with the paper's own cadence of 350 tokens and a prompt that is no multiple of the unit: rounds fire at
    # lengths with a short last unit, so the layers of a rollout keep different token counts (a length per list)
    8: dict(name="paper-math-ragged-B2048", L=28, Hq=12, Hkv=2, d=128, dtype="bf16", B=2048, T=337, n_protect=0,
            budget=10, block=32, lists=1, logit_std=1.0, steps=1050, cadence=350, outliers=0, data_seed=0, noise_seed=1,
            per_list_lens=True),
}
