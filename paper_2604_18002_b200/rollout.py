"""Rollout driver: owns the device buffers of a batch of rollouts and strings
the five library calls together (one eviction round, then decode steps).

Nothing here computes: every step is a call into the CUDA library through
``binding``; this module only allocates tensors, keeps the workspaces and
enqueues the calls on the current stream (no host synchronisation between
calls).  ``run_from_host`` is the host-buffer entry: it stages pinned host
inputs to the device on a copy stream, overlapped with the compute stream, and
streams the attention outputs back.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as ngc


class NgcRollout:
    def __init__(self, L, B, Hq, Hkv, d, dtype, capacity, n_max, k_max, lists=ngc.LISTS_SHARED, block=1,
                 w=5, device="cuda", list_base=0, with_score=True, kv=None, per_list_lens=False):
        """``kv``: optional (k, v) device tensors of shape [L][Hkv][sum(capacity)][d] to adopt
        instead of allocating fresh ones.  ``per_list_lens``: keep one cache length per (sequence,
        eviction list) instead of one per sequence, so that lists may keep different token counts
        (units of several tokens with a short last unit); needs ``lists`` != shared."""
        self.L, self.B, self.Hq, self.Hkv, self.d = L, B, Hq, Hkv, d
        self.dtype, self.lists, self.block, self.w = dtype, lists, block, w
        self.device = device
        self.list_base = list_base
        self.G = ngc.lists_G(lists, L, Hkv)
        cap = torch.as_tensor(capacity, dtype=torch.int64).expand(B).clone()
        seq_off = torch.zeros(B + 1, dtype=torch.int64)
        seq_off[1:] = torch.cumsum(cap, 0)
        R = int(seq_off[-1])
        if kv is None:
            kv = (torch.empty((L, Hkv, R, d), dtype=dtype, device=device),
                  torch.empty((L, Hkv, R, d), dtype=dtype, device=device))
        assert tuple(kv[0].shape) == (L, Hkv, R, d) and tuple(kv[1].shape) == (L, Hkv, R, d)
        lens_shape = (B, self.G) if per_list_lens else (B,)
        self.cache = ngc.NgcCache(kv[0], kv[1], seq_off.to(device), torch.zeros(lens_shape, dtype=torch.int32, device=device),
                                  Hq, int(cap.max()), lists if per_list_lens else 0)
        self.n_max, self.k_max = n_max, k_max
        self.logits = torch.empty((B, self.G, n_max), dtype=torch.float32, device=device)
        self.score_logits = torch.empty_like(self.logits) if with_score else None
        self.kept_order = torch.empty((B, self.G, k_max), dtype=torch.int32, device=device)
        self.kept_sorted = torch.empty((B, self.G, k_max), dtype=torch.int32, device=device)
        self.logp = torch.empty((1, B, self.G), dtype=torch.float64, device=device)
        self.n_units = torch.zeros((B,), dtype=torch.int32, device=device)     # written by ngc_score_evict
        self.status = ngc.new_status(device)
        self.ws_decode = ngc.alloc_workspace(ngc.workspace_bytes(ngc.OP_DECODE, self.cache), device)
        self.ws_sample = ngc.alloc_workspace(ngc.workspace_bytes(ngc.OP_SAMPLE, None, self.G, n_max, k_max, B=B), device)
        self.ws_score = ngc.alloc_workspace(ngc.workspace_bytes(ngc.OP_SCORE, self.cache, self.G, n_max), device) \
            if with_score else None
        self.launches = 0          # kernels enqueued so far (bookkeeping for the benchmark)

    # ---- one eviction round: score -> sample -> log-prob -> compact ----------------
    def eviction_round(self, n: torch.Tensor, n_protect: Optional[torch.Tensor], budget: torch.Tensor, seed: int,
                       rnd: int, q_recent: Optional[torch.Tensor] = None, logits: Optional[torch.Tensor] = None,
                       greedy: int = 0):
        """Samples from ``logits`` if given, else from the scores of ``q_recent``.  When both are
        given the scores are still computed (into ``score_logits``) but the draw uses ``logits``.
        With a cache length per list and a draw from the scores, ``n`` is ignored: the unit counts
        come from the scoring call."""
        if q_recent is not None:
            target = self.score_logits if logits is not None else self.logits
            ngc.ngc_score_evict(self.cache, q_recent, self.block, self.lists, target, ws=self.ws_score, status=self.status,
                                n_units_out=self.n_units)
            self.launches += ngc.score_launches(self.cache, q_recent.shape[3])
            if self.cache.lens_lists and logits is None:
                n = self.n_units        # a length per list: the library reports the unit count of each rollout's longest list
        src = logits if logits is not None else self.logits
        ngc.ngc_sample_evict(src, n, n_protect, budget, seed, rnd, self.kept_order, self.kept_sorted, None,
                             greedy=greedy, list_base=self.list_base, ws=self.ws_sample, status=self.status)
        ngc.ngc_evict_logprob(src, n, n_protect, budget, self.kept_order, self.logp, status=self.status)
        ngc.ngc_compact_kv(self.cache, self.kept_sorted, budget, self.lists, self.block, status=self.status)
        self.launches += 4 + (1 if self.G > 1 and not self.cache.lens_lists else 0)     # compaction's check kernel

    # ---- one decode step over all layers ------------------------------------------
    def decode_step(self, q: torch.Tensor, out: torch.Tensor, new_k: Optional[torch.Tensor] = None,
                    new_v: Optional[torch.Tensor] = None):
        ngc.ngc_decode_attn_ragged(self.cache, q, out, new_k, new_v, ws=self.ws_decode, status=self.status)
        split = ngc.decode_splits(self.cache, append=new_k is not None) > 1
        self.launches += 1 + (1 if new_k is not None else 0) + (1 if split else 0)

    def capture_decode_steps(self, q: torch.Tensor, out: torch.Tensor, new_k: torch.Tensor, new_v: torch.Tensor):
        """Records the decode calls of ``q.shape[0]`` consecutive steps (step s reads ``q[s]``, ``new_k[s]``,
        ``new_v[s]`` and writes ``out[s]``) into one CUDA graph and returns it; ``graph.replay()`` then runs all
        of them with a single launch from the host.  For short caches and small batches a decode step is a few
        microseconds of GPU work, less than the host needs to enqueue its kernels, so the loop is launch-bound
        unless it is replayed as a graph.  Call ``decode_step`` once before capturing (the first call of a
        process configures the kernels); the tensors must stay alive and in place while the graph is used."""
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for s in range(q.shape[0]):
                self.decode_step(q[s], out[s], new_k[s], new_v[s])
        return graph

    def check_status(self):
        code = int(self.status.item())
        if code != 0:
            raise ngc.NgcError(f"device status {code}: {ngc.DEV_STATUS.get(code, '?')}")


class HostStep:
    """Host-buffer driver for one whole step (eviction round + decode steps): pinned host
    inputs in, attention outputs and eviction results out, copies overlapped with compute.

    The K/V cache is by far the largest input.  With ``double_buffer=True`` the driver owns a
    second K/V pair on the device: ``run(..., prefetch_next=(h_k, h_v))`` uploads the NEXT
    step's cache into the spare pair on the copy stream while the current step computes, and
    the next ``run`` adopts that pair instead of waiting for its own upload."""

    def __init__(self, ro: NgcRollout, steps: int, chunk: int = 16, double_buffer: bool = False):
        self.ro, self.steps, self.chunk = ro, steps, chunk
        dev = ro.device
        L, B, Hq, Hkv, d = ro.L, ro.B, ro.Hq, ro.Hkv, ro.d
        self.d_q = torch.empty((steps, L, B, Hq, d), dtype=ro.dtype, device=dev)
        self.d_nk = torch.empty((steps, L, B, Hkv, d), dtype=ro.dtype, device=dev)
        self.d_nv = torch.empty_like(self.d_nk)
        self.d_out = torch.empty((steps, L, B, Hq, d), dtype=torch.float32, device=dev)
        self.copy_in = torch.cuda.Stream(device=dev)
        self.copy_out = torch.cuda.Stream(device=dev)
        self.spare = (torch.empty_like(ro.cache.k), torch.empty_like(ro.cache.v)) if double_buffer else None
        self.staged = None          # event: the spare pair holds the next step's cache

    def _stage_next(self, h_k, h_v):
        """Upload the next step's cache into the spare pair (copy stream); returns the bytes enqueued."""
        main = torch.cuda.current_stream()
        self.copy_in.wait_stream(main)      # the spare pair was the previous step's cache: its kernels must be done
        with torch.cuda.stream(self.copy_in):
            self.spare[0].copy_(h_k, non_blocking=True)
            self.spare[1].copy_(h_v, non_blocking=True)
            self.staged = torch.cuda.Event()
            self.staged.record(self.copy_in)
        return h_k.numel() * h_k.element_size() + h_v.numel() * h_v.element_size()

    def run(self, h_k, h_v, h_lens, h_logits, h_q, h_nk, h_nv, h_out, h_kept_order, h_logp, n, n_protect, budget,
            seed, rnd, h_q_recent=None, d_q_recent=None, prefetch_next=None):
        """All ``h_*`` are pinned host tensors.  Returns (h2d_bytes, d2h_bytes) enqueued by this call."""
        ro = self.ro
        main = torch.cuda.current_stream()
        h2d = 0
        d2h = 0
        if self.staged is not None:
            # this step's cache was uploaded during the previous step: adopt the pair, no copy now
            main.wait_event(self.staged)
            self.staged = None
            (ro.cache.k, ro.cache.v), self.spare = self.spare, (ro.cache.k, ro.cache.v)
            first = ((ro.cache.lens, h_lens), (ro.logits, h_logits))
        else:
            first = ((ro.cache.k, h_k), (ro.cache.v, h_v), (ro.cache.lens, h_lens), (ro.logits, h_logits))
        # what the eviction round needs first is copied on the compute stream
        for dst, src in first:
            dst.copy_(src, non_blocking=True)
            h2d += src.numel() * src.element_size()
        if h_q_recent is not None:
            d_q_recent.copy_(h_q_recent, non_blocking=True)
            h2d += h_q_recent.numel() * h_q_recent.element_size()
        # decode inputs stream in chunk by chunk on the copy stream
        self.copy_in.wait_stream(main)
        in_events = []
        with torch.cuda.stream(self.copy_in):
            for s0 in range(0, self.steps, self.chunk):
                s1 = min(self.steps, s0 + self.chunk)
                for dst, src in ((self.d_q, h_q), (self.d_nk, h_nk), (self.d_nv, h_nv)):
                    dst[s0:s1].copy_(src[s0:s1], non_blocking=True)
                    h2d += src[s0:s1].numel() * src.element_size()
                ev = torch.cuda.Event()
                ev.record(self.copy_in)
                in_events.append(ev)
        if prefetch_next is not None and self.spare is not None:
            h2d += self._stage_next(*prefetch_next)          # behind this step's decode inputs on the copy stream
        ro.eviction_round(n, n_protect, budget, seed, rnd, q_recent=d_q_recent, logits=ro.logits)
        h_kept_order.copy_(ro.kept_order, non_blocking=True)
        h_logp.copy_(ro.logp, non_blocking=True)
        d2h += ro.kept_order.numel() * 4 + ro.logp.numel() * 8
        for ci, s0 in enumerate(range(0, self.steps, self.chunk)):
            s1 = min(self.steps, s0 + self.chunk)
            main.wait_event(in_events[ci])
            for s in range(s0, s1):
                ro.decode_step(self.d_q[s], self.d_out[s], self.d_nk[s], self.d_nv[s])
            ev = torch.cuda.Event()
            ev.record(main)
            self.copy_out.wait_event(ev)
            with torch.cuda.stream(self.copy_out):
                h_out[s0:s1].copy_(self.d_out[s0:s1], non_blocking=True)
            d2h += self.d_out[s0:s1].numel() * 4
        main.wait_stream(self.copy_out)
        return h2d, d2h
