"""Thin Python binding of the C-ABI CUDA library (``include/ngc.h``).

Argument marshalling only: torch tensors provide device memory and the current
CUDA stream, every step of the path runs inside the library's kernels.  There
is no CPU fallback: importing this module without the built library raises,
and so does every call made without a CUDA device.
"""
from __future__ import annotations

import contextlib
import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libngc_b200.so")

F32, BF16 = 0, 1
LISTS_SHARED, LISTS_PER_LAYER, LISTS_PER_LAYER_KVHEAD = 0, 1, 2
OP_SCORE, OP_SAMPLE, OP_LOGPROB, OP_COMPACT, OP_DECODE, OP_SCORE_BACKWARD = range(6)

DEV_STATUS = {0: "ok", 1: "bad counts", 2: "NaN logit", 3: "bad kept list", 4: "strip full",
              5: "lists disagree", 6: "timeout", 7: "index out of bounds (bounds-checking build)"}

EXPORTS = ["ngc_version", "ngc_strerror", "ngc_last_cuda_error", "ngc_workspace_bytes", "ngc_decode_splits", "ngc_score_evict", "ngc_score_evict_launches",
           "ngc_sample_evict", "ngc_evict_logprob", "ngc_evict_logprob_backward", "ngc_compact_kv", "ngc_decode_attn_ragged",
           "ngc_decode_attn_ragged_static", "ngc_evict_pages", "ngc_decode_attn_paged", "ngc_score_evict_paged", "ngc_replay_visibility", "ngc_score_evict_backward", "ngc_replay_attn", "ngc_replay_attn_variant", "ngc_selftest_bounded_wait"]
STATIC_SCRATCH_BYTES = 8 << 20


class NgcError(RuntimeError):
    pass


class CacheDesc(C.Structure):
    """Mirror of ``ngc_cache``."""
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("seq_off", C.c_void_p), ("lens", C.c_void_p),
                ("rows", C.c_int64), ("L", C.c_int32), ("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
                ("d", C.c_int32), ("dtype", C.c_int32), ("max_len", C.c_int32), ("lens_lists", C.c_int32)]


class PagedCacheDesc(C.Structure):
    """Mirror of ``ngc_paged_cache``."""
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("page_table", C.c_void_p), ("lens", C.c_void_p),
                ("L", C.c_int32), ("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32),
                ("dtype", C.c_int32), ("page", C.c_int32), ("pages_cap", C.c_int32), ("lists", C.c_int32),
                ("lens_per_list", C.c_int32)]


def _load(path: str = LIB_PATH):
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2604_18002_b200.build` "
            "(there is no CPU fallback)")
    lib = C.CDLL(path)
    vp, i32, u32, u64, sz = C.c_void_p, C.c_int, C.c_uint32, C.c_uint64, C.c_size_t
    lib.ngc_version.restype = i32
    lib.ngc_strerror.restype = C.c_char_p
    lib.ngc_strerror.argtypes = [i32]
    lib.ngc_last_cuda_error.restype = i32
    lib.ngc_workspace_bytes.restype = sz
    lib.ngc_workspace_bytes.argtypes = [i32, C.POINTER(CacheDesc), i32, i32, i32]
    lib.ngc_decode_splits.restype = i32
    lib.ngc_decode_splits.argtypes = [C.POINTER(CacheDesc), i32]
    lib.ngc_score_evict_launches.restype = i32
    lib.ngc_score_evict_launches.argtypes = [C.POINTER(CacheDesc), i32]
    lib.ngc_score_evict.restype = i32
    lib.ngc_score_evict.argtypes = [C.POINTER(CacheDesc), vp, i32, i32, i32, i32, vp, i32, vp, vp, sz, vp, vp]
    lib.ngc_sample_evict.restype = i32
    lib.ngc_sample_evict.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, u64, u64, u32, i32, vp, vp, vp, vp, sz, vp, vp]
    lib.ngc_evict_logprob.restype = i32
    lib.ngc_evict_logprob.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, sz, vp, vp]
    lib.ngc_evict_logprob_backward.restype = i32
    lib.ngc_evict_logprob_backward.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, sz, vp, vp]
    lib.ngc_compact_kv.restype = i32
    lib.ngc_compact_kv.argtypes = [C.POINTER(CacheDesc), vp, vp, i32, i32, i32, vp, vp]
    lib.ngc_decode_attn_ragged.restype = i32
    lib.ngc_decode_attn_ragged.argtypes = [C.POINTER(CacheDesc), vp, vp, vp, i32, i32, C.c_float, vp, i32, vp, sz, vp, vp]
    lib.ngc_decode_attn_ragged_static.restype = i32
    lib.ngc_decode_attn_ragged_static.argtypes = [C.POINTER(CacheDesc), vp, vp, vp, i32, i32, C.c_float, vp, i32, vp, vp]
    lib.ngc_score_evict_paged.restype = i32
    lib.ngc_score_evict_paged.argtypes = [C.POINTER(PagedCacheDesc), vp, i32, i32, vp, i32, vp, vp, sz, vp, vp]
    lib.ngc_score_evict_backward.restype = i32
    lib.ngc_score_evict_backward.argtypes = [C.POINTER(CacheDesc), vp, i32, i32, i32, i32, vp, vp, i32, vp, vp, vp, sz, vp, vp]
    lib.ngc_replay_attn.restype = i32
    lib.ngc_replay_attn.argtypes = [C.POINTER(CacheDesc), vp, i32, vp, vp, vp, i32, i32, i32, C.c_float, vp, i32, vp, vp]
    lib.ngc_replay_attn_variant.restype = i32
    lib.ngc_replay_attn_variant.argtypes = [C.POINTER(CacheDesc), vp, i32, vp, vp, vp, i32, i32, i32, C.c_float, vp, i32, i32, vp, vp]
    lib.ngc_replay_visibility.restype = i32
    lib.ngc_replay_visibility.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.ngc_selftest_bounded_wait.restype = i32
    lib.ngc_selftest_bounded_wait.argtypes = [u32, vp, vp, vp]
    lib.ngc_evict_pages.restype = i32
    lib.ngc_evict_pages.argtypes = [C.POINTER(PagedCacheDesc), vp, vp, i32, vp, vp]
    lib.ngc_decode_attn_paged.restype = i32
    lib.ngc_decode_attn_paged.argtypes = [C.POINTER(PagedCacheDesc), vp, vp, vp, i32, i32, C.c_float, vp, i32, vp, sz, vp, vp]
    return lib


lib = _load()


@contextlib.contextmanager
def use_library(path: str):
    """Route every call of this module to another build of the library (the bounds-checking or the
    NVTX build) for the duration of the block."""
    global lib
    saved, lib = lib, _load(path)
    try:
        yield lib
    finally:
        lib = saved


def _check(rc: int, what: str):
    if rc != 0:
        msg = lib.ngc_strerror(rc).decode()
        if rc == -4:
            msg += f" (cudaError {lib.ngc_last_cuda_error()})"
        raise NgcError(f"{what}: {msg}")


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise NgcError("device tensors required: the library has no CPU path")
    if not t.is_contiguous():
        raise NgcError("contiguous tensors required")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise NgcError(f"unsupported cache dtype {t.dtype}")


def lists_G(lists: int, L: int, Hkv: int) -> int:
    return 1 if lists == LISTS_SHARED else (L if lists == LISTS_PER_LAYER else L * Hkv)


@dataclass
class NgcCache:
    """Device K/V cache plus the host-side numbers the launches need."""
    k: torch.Tensor        # [L][Hkv][R][d]
    v: torch.Tensor
    seq_off: torch.Tensor  # int64 [B+1], device
    lens: torch.Tensor     # int32 [B] (or [B][G] with lens_lists != 0), device
    Hq: int
    max_len: int           # host bound on lens (any value >= max(lens) at call time)
    lens_lists: int = 0    # 0: one length per sequence; LISTS_PER_LAYER / _KVHEAD: one per (sequence, list)

    def desc(self, extra_len: int = 0) -> CacheDesc:
        L, Hkv, R, d = self.k.shape
        if self.lens_lists:
            assert tuple(self.lens.shape) == (self.seq_off.shape[0] - 1, lists_G(self.lens_lists, L, Hkv))
        return CacheDesc(_ptr(self.k), _ptr(self.v), _ptr(self.seq_off), _ptr(self.lens), R, L,
                         self.seq_off.shape[0] - 1, self.Hq, Hkv, d, _dtype_code(self.k), self.max_len + extra_len,
                         self.lens_lists)

    @property
    def L(self):
        return self.k.shape[0]

    @property
    def B(self):
        return self.seq_off.shape[0] - 1

    @property
    def Hkv(self):
        return self.k.shape[1]

    @property
    def d(self):
        return self.k.shape[3]


def version() -> int:
    return lib.ngc_version()


def workspace_bytes(op: int, cache: Optional[NgcCache] = None, G: int = 1, n_max: int = 0, k_max: int = 0,
                    B: Optional[int] = None) -> int:
    if cache is not None:
        d = cache.desc(1)
    else:
        d = CacheDesc(None, None, None, None, 0, 1, B or 1, 1, 1, 128, BF16, 0)
    return int(lib.ngc_workspace_bytes(op, C.byref(d), G, n_max, k_max))


def decode_splits(cache: NgcCache, layers: Optional[int] = None, append: bool = True) -> int:
    d = cache.desc(1 if append else 0)
    return int(lib.ngc_decode_splits(C.byref(d), cache.L if layers is None else layers))


def score_launches(cache: NgcCache, w: int) -> int:
    """Kernels one ngc_score_evict call enqueues (launch counting)."""
    d = cache.desc()
    return int(lib.ngc_score_evict_launches(C.byref(d), w))


def alloc_workspace(nbytes: int, device="cuda") -> Optional[torch.Tensor]:
    if nbytes == 0:
        return None
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


def ngc_score_evict(cache: NgcCache, q_recent: torch.Tensor, block: int, lists: int, logits: torch.Tensor,
                    log_transform: int = 0, ws: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                    n_units_out: Optional[torch.Tensor] = None):
    """q_recent [L][B][Hq][w][d] -> logits [B][G][n_max] fp32 (in place); n_units_out int32 [B] (optional):
    the unit count per sequence to hand to the sampler."""
    w = q_recent.shape[3]
    n_max = logits.shape[2]
    d = cache.desc()
    rc = lib.ngc_score_evict(C.byref(d), _ptr(q_recent), w, block, lists, log_transform, _ptr(logits), n_max,
                             _ptr(n_units_out), _ptr(ws), 0 if ws is None else ws.numel(), _ptr(status), _stream())
    _check(rc, "ngc_score_evict")


def ngc_sample_evict(logits: torch.Tensor, n: torch.Tensor, n_protect: Optional[torch.Tensor], budget: torch.Tensor,
                     seed: int, rnd: int, kept_order: torch.Tensor, kept_sorted: torch.Tensor,
                     keep_mask: Optional[torch.Tensor] = None, greedy: int = 0, list_base: int = 0,
                     ws: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None):
    B, G, n_max = logits.shape
    k_max = kept_order.shape[2]
    rc = lib.ngc_sample_evict(_ptr(logits), _ptr(n), _ptr(n_protect), _ptr(budget), B, G, n_max, k_max,
                              seed, rnd, list_base, greedy, _ptr(kept_order), _ptr(kept_sorted), _ptr(keep_mask),
                              _ptr(ws), 0 if ws is None else ws.numel(), _ptr(status), _stream())
    _check(rc, "ngc_sample_evict")


def ngc_evict_logprob(logits: torch.Tensor, n: torch.Tensor, n_protect: Optional[torch.Tensor], budget: torch.Tensor,
                      kept_order: torch.Tensor, logp: torch.Tensor, status: Optional[torch.Tensor] = None):
    """logits [NB][B][G][n_max] (or [B][G][n_max]); logp fp64 [NB][B][G]."""
    if logits.dim() == 3:
        NB = 1
        B, G, n_max = logits.shape
    else:
        NB, B, G, n_max = logits.shape
    k_max = kept_order.shape[-1]
    rc = lib.ngc_evict_logprob(_ptr(logits), _ptr(n), _ptr(n_protect), _ptr(budget), _ptr(kept_order),
                               NB, B, G, n_max, k_max, _ptr(logp), None, 0, _ptr(status), _stream())
    _check(rc, "ngc_evict_logprob")


def ngc_evict_logprob_backward(logits: torch.Tensor, n: torch.Tensor, n_protect: Optional[torch.Tensor], budget: torch.Tensor,
                               kept_order: torch.Tensor, grad_logits: torch.Tensor, grad_logp: Optional[torch.Tensor] = None,
                               status: Optional[torch.Tensor] = None):
    """grad_logits fp32, same shape as logits; grad_logp fp64 [NB][B][G] or None (= ones)."""
    if logits.dim() == 3:
        NB = 1
        B, G, n_max = logits.shape
    else:
        NB, B, G, n_max = logits.shape
    k_max = kept_order.shape[-1]
    rc = lib.ngc_evict_logprob_backward(_ptr(logits), _ptr(n), _ptr(n_protect), _ptr(budget), _ptr(kept_order), _ptr(grad_logp),
                                        NB, B, G, n_max, k_max, _ptr(grad_logits), None, 0, _ptr(status), _stream())
    _check(rc, "ngc_evict_logprob_backward")


def ngc_compact_kv(cache: NgcCache, kept_sorted: torch.Tensor, budget: torch.Tensor, lists: int, block: int = 1,
                   status: Optional[torch.Tensor] = None):
    d = cache.desc()
    rc = lib.ngc_compact_kv(C.byref(d), _ptr(kept_sorted), _ptr(budget), kept_sorted.shape[2], lists, block,
                            _ptr(status), _stream())
    _check(rc, "ngc_compact_kv")


def ngc_decode_attn_ragged(cache: NgcCache, q: torch.Tensor, out: torch.Tensor, new_k: Optional[torch.Tensor] = None,
                           new_v: Optional[torch.Tensor] = None, layer_begin: int = 0, layer_end: Optional[int] = None,
                           scale: Optional[float] = None, ws: Optional[torch.Tensor] = None,
                           status: Optional[torch.Tensor] = None):
    if layer_end is None:
        layer_end = cache.L
    if scale is None:
        scale = 1.0 / (cache.d ** 0.5)
    d = cache.desc(1 if new_k is not None else 0)
    rc = lib.ngc_decode_attn_ragged(C.byref(d), _ptr(q), _ptr(new_k), _ptr(new_v), layer_begin, layer_end,
                                    scale, _ptr(out), _dtype_code(out), _ptr(ws), 0 if ws is None else ws.numel(),
                                    _ptr(status), _stream())
    _check(rc, "ngc_decode_attn_ragged")


def ngc_decode_attn_ragged_static(cache: NgcCache, q: torch.Tensor, out: torch.Tensor, new_k: Optional[torch.Tensor] = None,
                                  new_v: Optional[torch.Tensor] = None, layer_begin: int = 0,
                                  layer_end: Optional[int] = None, scale: Optional[float] = None,
                                  status: Optional[torch.Tensor] = None):
    """Decode attention for callers that cannot supply device scratch memory: the split partials
    live in an array built into the library (``STATIC_SCRATCH_BYTES``), nothing is allocated.
    Keep calls stream-ordered (they share the array); make the first call on a device outside
    any stream capture (it looks the array's address up).  Raises when the launch would need
    more scratch than the array holds."""
    if layer_end is None:
        layer_end = cache.L
    if scale is None:
        scale = 1.0 / (cache.d ** 0.5)
    d = cache.desc(1 if new_k is not None else 0)
    rc = lib.ngc_decode_attn_ragged_static(C.byref(d), _ptr(q), _ptr(new_k), _ptr(new_v), layer_begin, layer_end,
                                           scale, _ptr(out), _dtype_code(out), _ptr(status), _stream())
    _check(rc, "ngc_decode_attn_ragged_static")


@dataclass
class NgcPagedCache:
    """Paged device K/V cache: one eviction unit = one page; eviction edits ``page_table`` only."""
    k: torch.Tensor           # [L][Hkv][B * pages_cap][page][d] bf16
    v: torch.Tensor
    page_table: torch.Tensor  # int32 [B][G][pages_cap], each row a permutation of 0..pages_cap-1
    lens: torch.Tensor        # int32 [B], or [B][G] (a length per list)
    Hq: int
    lists: int

    def desc(self) -> PagedCacheDesc:
        L, Hkv, n_pages, page, d = self.k.shape
        B, G, pages_cap = self.page_table.shape
        assert n_pages == B * pages_cap and G == lists_G(self.lists, L, Hkv)
        return PagedCacheDesc(_ptr(self.k), _ptr(self.v), _ptr(self.page_table), _ptr(self.lens), L, B, self.Hq, Hkv, d,
                              _dtype_code(self.k), page, pages_cap, self.lists, 1 if self.lens.dim() == 2 else 0)

    def as_contiguous_desc(self) -> "NgcCache":
        """Shape-only view for workspace sizing (same L, B, Hq, Hkv)."""
        L, Hkv, n_pages, page, d = self.k.shape
        B, _, pages_cap = self.page_table.shape
        flat = self.k.view(L, Hkv, n_pages * page, d)
        return NgcCache(flat, flat, torch.zeros(B + 1, dtype=torch.int64, device=self.k.device), self.lens, self.Hq, pages_cap * page)


def ngc_evict_pages(cache: NgcPagedCache, kept_sorted: torch.Tensor, budget: torch.Tensor, status: Optional[torch.Tensor] = None):
    d = cache.desc()
    rc = lib.ngc_evict_pages(C.byref(d), _ptr(kept_sorted), _ptr(budget), kept_sorted.shape[2], _ptr(status), _stream())
    _check(rc, "ngc_evict_pages")


def ngc_decode_attn_paged(cache: NgcPagedCache, q: torch.Tensor, out: torch.Tensor, new_k: Optional[torch.Tensor] = None,
                          new_v: Optional[torch.Tensor] = None, layer_begin: int = 0, layer_end: Optional[int] = None,
                          scale: Optional[float] = None, ws: Optional[torch.Tensor] = None,
                          status: Optional[torch.Tensor] = None):
    L, d = cache.k.shape[0], cache.k.shape[4]
    if layer_end is None:
        layer_end = L
    if scale is None:
        scale = 1.0 / (d ** 0.5)
    desc = cache.desc()
    rc = lib.ngc_decode_attn_paged(C.byref(desc), _ptr(q), _ptr(new_k), _ptr(new_v), layer_begin, layer_end, scale,
                                   _ptr(out), _dtype_code(out), _ptr(ws), 0 if ws is None else ws.numel(), _ptr(status), _stream())
    _check(rc, "ngc_decode_attn_paged")


def ngc_score_evict_paged(cache: NgcPagedCache, q_recent: torch.Tensor, logits: torch.Tensor, log_transform: int = 0,
                          ws: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                          n_units_out: Optional[torch.Tensor] = None):
    """q_recent [L][B][Hq][w][d] -> logits [B][G][n_max] fp32 (units = pages)."""
    d = cache.desc()
    rc = lib.ngc_score_evict_paged(C.byref(d), _ptr(q_recent), q_recent.shape[3], log_transform, _ptr(logits), logits.shape[2],
                                   _ptr(n_units_out), _ptr(ws), 0 if ws is None else ws.numel(), _ptr(status), _stream())
    _check(rc, "ngc_score_evict_paged")


def ngc_replay_visibility(kept_sorted: torch.Tensor, budget: torch.Tensor, alive_before: torch.Tensor, total_before: torch.Tensor,
                          block: int, alive_max: int, alive_pos: torch.Tensor, alive_count: torch.Tensor,
                          status: Optional[torch.Tensor] = None):
    """kept_sorted [R][B][G][k_max] -> alive_pos [R][B][G][k_max*block], alive_count [R][B][G] (int32)."""
    R, B, G, k_max = kept_sorted.shape
    rc = lib.ngc_replay_visibility(_ptr(kept_sorted), _ptr(budget), _ptr(alive_before), _ptr(total_before), R, B, G, k_max, block,
                                   alive_max, 1 if alive_before.dim() == 3 else 0, _ptr(alive_pos), _ptr(alive_count), _ptr(status),
                                   _stream())
    _check(rc, "ngc_replay_visibility")


def ngc_score_evict_backward(cache: NgcCache, q_recent: torch.Tensor, block: int, lists: int, grad_logits: torch.Tensor,
                             grad_q_recent: torch.Tensor, grad_k: torch.Tensor, logits: Optional[torch.Tensor] = None,
                             log_transform: int = 0, ws: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None):
    """grad_logits [B][G][n_max] fp32 -> grad_q_recent fp32 (shape of q_recent), grad_k (shape and dtype of cache.k)."""
    d = cache.desc()
    rc = lib.ngc_score_evict_backward(C.byref(d), _ptr(q_recent), q_recent.shape[3], block, lists, log_transform, _ptr(logits),
                                      _ptr(grad_logits), grad_logits.shape[2], _ptr(grad_q_recent), _ptr(grad_k),
                                      _ptr(ws), 0 if ws is None else ws.numel(), _ptr(status), _stream())
    _check(rc, "ngc_score_evict_backward")


REPLAY_ATTN_AUTO, REPLAY_ATTN_MMA_SYNC, REPLAY_ATTN_TCGEN05 = 0, 1, 2


def ngc_replay_attn(cache: NgcCache, q: torch.Tensor, out: torch.Tensor, alive_pos: Optional[torch.Tensor] = None,
                    alive_count: Optional[torch.Tensor] = None, total_before: Optional[torch.Tensor] = None,
                    lists: int = LISTS_SHARED, scale: Optional[float] = None, status: Optional[torch.Tensor] = None,
                    variant: Optional[int] = None):
    """q, out [L][B][Hq][t_max][d]; cache holds the full sequences (lens = total tokens).  ``variant`` picks the device
    path (REPLAY_ATTN_*) through ngc_replay_attn_variant; None calls ngc_replay_attn itself."""
    t_max = q.shape[3]
    if scale is None:
        scale = 1.0 / (cache.d ** 0.5)
    n_rounds = 0 if alive_pos is None else alive_pos.shape[0]
    kt_max = 0 if alive_pos is None else alive_pos.shape[3]
    d = cache.desc()
    if variant is None:
        rc = lib.ngc_replay_attn(C.byref(d), _ptr(q), t_max, _ptr(alive_pos), _ptr(alive_count), _ptr(total_before), n_rounds, kt_max,
                                 lists, scale, _ptr(out), _dtype_code(out), _ptr(status), _stream())
    else:
        rc = lib.ngc_replay_attn_variant(C.byref(d), _ptr(q), t_max, _ptr(alive_pos), _ptr(alive_count), _ptr(total_before), n_rounds,
                                         kt_max, lists, scale, _ptr(out), _dtype_code(out), variant, _ptr(status), _stream())
    _check(rc, "ngc_replay_attn")


def ngc_selftest_bounded_wait(limit_us: int, status: torch.Tensor, waited_ns: Optional[torch.Tensor] = None):
    """One warp waits at most ``limit_us`` microseconds on a barrier that never completes; ``status`` becomes the
    timeout code and the call returns normally (diagnostic of the kernels' bounded waits)."""
    rc = lib.ngc_selftest_bounded_wait(limit_us, _ptr(status), _ptr(waited_ns), _stream())
    _check(rc, "ngc_selftest_bounded_wait")
