"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE ONLY).

The oracle is a plain C++ restatement of the paper's definitions (Sections
4.1-4.3).  Only the test suite, the smoke check and the CPU-baseline leg of the
benchmark may import this package; the CUDA library never does, and this
package never imports the CUDA library.

Arrays are numpy, host memory.  bfloat16 data is passed as ``uint16`` bit
patterns (``dtype=1``); fp32 as ``float32`` (``dtype=0``).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ngc_oracle.cpp")
_HDR = os.path.join(_HERE, "ngc_oracle.h")
_SO = os.path.join(_HERE, "libngc_oracle.so")

F32, BF16 = 0, 1
LISTS_SHARED, LISTS_PER_LAYER, LISTS_PER_LAYER_KVHEAD = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    stale = (not os.path.exists(_SO)) or any(
        os.path.getmtime(p) > os.path.getmtime(_SO) for p in (_SRC, _HDR))
    if force or stale:
        tmp = _SO + f".tmp{os.getpid()}"
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", tmp, _SRC]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ngc_oracle_dlog.restype = C.c_float
        _lib.ngc_oracle_dlog.argtypes = [C.c_float]
        _lib.ngc_oracle_uniform.restype = C.c_float
        _lib.ngc_oracle_uniform.argtypes = [C.c_uint32]
        _lib.ngc_oracle_gumbel.restype = C.c_float
        _lib.ngc_oracle_gumbel.argtypes = [C.c_uint32]
        _lib.ngc_oracle_perturbed_key.restype = C.c_float
        _lib.ngc_oracle_perturbed_key.argtypes = [C.c_float, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def lists_G(lists: int, L: int, Hkv: int) -> int:
    return 1 if lists == LISTS_SHARED else (L if lists == LISTS_PER_LAYER else L * Hkv)


def threads() -> int:
    return int(lib().ngc_oracle_threads())


def philox4x32_10(ctr, key) -> np.ndarray:
    ctr = _c(ctr, np.uint32)
    key = _c(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().ngc_oracle_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def dlog(x: float) -> float:
    return float(lib().ngc_oracle_dlog(C.c_float(x)))


def uniform(x: int) -> float:
    return float(lib().ngc_oracle_uniform(C.c_uint32(x)))


def gumbel(x: int) -> float:
    return float(lib().ngc_oracle_gumbel(C.c_uint32(x)))


def perturbed_key(logit, seed, rnd, lst, i, greedy=0) -> float:
    return float(lib().ngc_oracle_perturbed_key(C.c_float(logit), seed, rnd, lst, i, greedy))


def sample_evict(logits, n, n_protect, budget, k_max, seed, rnd, greedy=0, list_base=0):
    """logits [B][G][n_max] fp32 -> (kept_order, kept_sorted, keep_mask, status)."""
    logits = _c(logits, np.float32)
    B, G, n_max = logits.shape
    n = _c(n, np.int32)
    budget = _c(budget, np.int32)
    n_protect = None if n_protect is None else _c(n_protect, np.int32)
    ko = np.empty((B, G, k_max), np.int32)
    ks = np.empty((B, G, k_max), np.int32)
    km = np.empty((B, G, n_max), np.uint8)
    st = np.zeros((B, G), np.int32)
    lib().ngc_oracle_sample_evict(_p(logits), _p(n), _p(n_protect), _p(budget), B, G, n_max, k_max,
                                  C.c_uint64(seed), C.c_uint64(rnd), C.c_uint32(list_base), int(greedy),
                                  _p(ko), _p(ks), _p(km), _p(st))
    return ko, ks, km, st


def _logprob(fn, logits, n, n_protect, budget, kept_order):
    logits = _c(logits, np.float32)
    if logits.ndim == 3:
        logits = logits[None]
    NB, B, G, n_max = logits.shape
    kept_order = _c(kept_order, np.int32).reshape(NB, B, G, -1)
    k_max = kept_order.shape[-1]
    n = _c(np.broadcast_to(np.asarray(n, np.int32).reshape(-1, B), (NB, B)), np.int32)
    budget = _c(np.broadcast_to(np.asarray(budget, np.int32).reshape(-1, B), (NB, B)), np.int32)
    if n_protect is not None:
        n_protect = _c(np.broadcast_to(np.asarray(n_protect, np.int32).reshape(-1, B), (NB, B)), np.int32)
    out = np.empty((NB, B, G), np.float64)
    rc = fn(_p(logits), _p(n), _p(n_protect), _p(budget), _p(kept_order), NB, B, G, n_max, k_max, _p(out))
    return out, rc


def evict_logprob(logits, n, n_protect, budget, kept_order):
    """Eq. (1) evaluated literally.  Returns (logp [NB][B][G] float64, rc)."""
    return _logprob(lib().ngc_oracle_evict_logprob, logits, n, n_protect, budget, kept_order)


def evict_logprob_scan(logits, n, n_protect, budget, kept_order):
    return _logprob(lib().ngc_oracle_evict_logprob_scan, logits, n, n_protect, budget, kept_order)


def evict_logprob_grad(logits, n, n_protect, budget, kept_order, grad_logp=None):
    """d logp / d logits from Eq. (1), term by term.  Returns (grad [NB][B][G][n_max] float64, rc)."""
    logits = _c(logits, np.float32)
    if logits.ndim == 3:
        logits = logits[None]
    NB, B, G, n_max = logits.shape
    kept_order = _c(kept_order, np.int32).reshape(NB, B, G, -1)
    k_max = kept_order.shape[-1]
    n = _c(np.broadcast_to(np.asarray(n, np.int32).reshape(-1, B), (NB, B)), np.int32)
    budget = _c(np.broadcast_to(np.asarray(budget, np.int32).reshape(-1, B), (NB, B)), np.int32)
    if n_protect is not None:
        n_protect = _c(np.broadcast_to(np.asarray(n_protect, np.int32).reshape(-1, B), (NB, B)), np.int32)
    if grad_logp is not None:
        grad_logp = _c(np.broadcast_to(np.asarray(grad_logp, np.float64), (NB, B, G)), np.float64)
    out = np.empty((NB, B, G, n_max), np.float64)
    rc = lib().ngc_oracle_evict_logprob_grad(_p(logits), _p(n), _p(n_protect), _p(budget), _p(kept_order), _p(grad_logp),
                                             NB, B, G, n_max, k_max, _p(out))
    return out, rc


def _dtype_of(a) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"cache arrays must be float32 or uint16 (bf16 bits), got {a.dtype}")


def compact_kv(k, v, seq_off, lens, kept_sorted, budget, lists, block=1):
    """k, v [L][Hkv][R][d].  Returns (k_out, v_out, new_lens, rc); rows beyond new_lens are zero."""
    L, Hkv, R, d = k.shape
    dt = _dtype_of(k)
    k = np.ascontiguousarray(k)
    v = np.ascontiguousarray(v)
    seq_off = _c(seq_off, np.int64)
    lens = _c(lens, np.int32)
    B = lens.shape[0]
    kept_sorted = _c(kept_sorted, np.int32)
    k_max = kept_sorted.shape[-1]
    budget = _c(budget, np.int32)
    ko = np.zeros_like(k)
    vo = np.zeros_like(v)
    nl = np.zeros(B, np.int32)
    rc = lib().ngc_oracle_compact_kv(_p(k), _p(v), _p(seq_off), _p(lens), L, B, Hkv, d, dt,
                                     _p(kept_sorted), _p(budget), k_max, int(lists), int(block),
                                     _p(ko), _p(vo), _p(nl))
    return ko, vo, nl, rc


def decode_attn(k, v, seq_off, lens, q, new_k=None, new_v=None, layer_begin=0, layer_end=None, scale=None):
    """In place on k, v, lens (append).  q [L][B][Hq][d].  Returns (out float64 [L][B][Hq][d], rc)."""
    L, Hkv, R, d = k.shape
    dt = _dtype_of(k)
    assert k.flags.c_contiguous and v.flags.c_contiguous and lens.dtype == np.int32
    seq_off = _c(seq_off, np.int64)
    B = lens.shape[0]
    Hq = q.shape[2]
    q = np.ascontiguousarray(q)
    assert _dtype_of(q) == dt
    if new_k is not None:
        new_k = np.ascontiguousarray(new_k)
        new_v = np.ascontiguousarray(new_v)
    if layer_end is None:
        layer_end = L
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((L, B, Hq, d), np.float64)
    rc = lib().ngc_oracle_decode_attn(_p(k), _p(v), _p(seq_off), _p(lens), L, B, Hq, Hkv, d, dt,
                                      _p(q), _p(new_k), _p(new_v), int(layer_begin), int(layer_end),
                                      C.c_double(scale), _p(out))
    return out, rc


def score_evict(k, seq_off, lens, q_recent, block, lists, log_transform=0, n_max=None):
    """q_recent [L][B][Hq][w][d].  Returns logits float64 [B][G][n_max] (NaN where no unit)."""
    L, Hkv, R, d = k.shape
    dt = _dtype_of(k)
    k = np.ascontiguousarray(k)
    seq_off = _c(seq_off, np.int64)
    lens = _c(lens, np.int32)
    B = lens.shape[0]
    q_recent = np.ascontiguousarray(q_recent)
    assert _dtype_of(q_recent) == dt
    Hq, w = q_recent.shape[2], q_recent.shape[3]
    G = lists_G(lists, L, Hkv)
    if n_max is None:
        n_max = int((int(lens.max()) + block - 1) // block) if B else 0
    out = np.full((B, G, n_max), np.nan, np.float64)
    lib().ngc_oracle_score_evict(_p(k), _p(seq_off), _p(lens), L, B, Hq, Hkv, d, dt,
                                 _p(q_recent), int(w), int(block), int(lists), int(log_transform),
                                 _p(out), int(n_max))
    return out


def score_evict_grad(k, seq_off, lens, q_recent, block, lists, grad_logits, log_transform=0):
    """Gradient of the scores w.r.t. q_recent and k.  grad_logits [B][G][n_max] float64.
    Returns (grad_q [L][B][Hq][w][d], grad_k [L][Hkv][R][d]) float64."""
    L, Hkv, R, d = k.shape
    dt = _dtype_of(k)
    k = np.ascontiguousarray(k)
    seq_off = _c(seq_off, np.int64)
    lens = _c(lens, np.int32)
    B = lens.shape[0]
    q_recent = np.ascontiguousarray(q_recent)
    assert _dtype_of(q_recent) == dt
    Hq, w = q_recent.shape[2], q_recent.shape[3]
    grad_logits = _c(grad_logits, np.float64)
    n_max = grad_logits.shape[2]
    gq = np.zeros((L, B, Hq, w, d), np.float64)
    gk = np.zeros((L, Hkv, R, d), np.float64)
    rc = lib().ngc_oracle_score_evict_grad(_p(k), _p(seq_off), _p(lens), L, B, Hq, Hkv, d, dt, _p(q_recent), w, int(block),
                                           int(lists), int(log_transform), _p(grad_logits), n_max, _p(gq), _p(gk))
    assert rc == 0
    return gq, gk
