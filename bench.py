"""Benchmark of the NGC hot path on B200.

One "step" = one pass of the whole hot path over one batch of synthetic
rollouts: an eviction round (score -> Gumbel-top-k sample -> log-prob ->
in-place compaction) followed by the workload's decode steps (append + ragged
attention over the surviving cache).  The workload is the 1.5B-shaped GQA
rollout step at B = 64: 28 layers, 12 query / 2 KV heads, d = 128, bf16 K/V,
4096 cached tokens evicted to 2048, then 256 decode steps.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ngc|reference]

With --gpus N > 1 and no rank environment, the script starts its own N ranks
(one process per GPU under torch.distributed.run on 127.0.0.1); started under
torchrun it takes the ranks it is given.  The batch of N x 64 rollouts is cut
into contiguous shards, one per rank, with no data-path collective.

Prints ONE JSON line (rank 0).  `value` is tokens/s with all inputs resident in
HBM; `e2e` is the same step driven from pinned host buffers through the public
host entry (copies inside the timed region); `roofline` is the decode kernel's
achieved HBM bandwidth, `compact` the compaction kernel's, `per_call_ms` the
time of each of the five calls; `config3` (one GPU only) repeats the per-call
figures on the 7B-shaped ragged batch; `cpu_baseline` is the CPU oracle timed
on a bounded sample of the same workload.

Measurement aids on one GPU (not the benchmark line):
    python bench.py --config 1|3|4|5|6|7 [--paged] [--graph]   per-phase timing of the other workloads
    python bench.py --kernel score_backward|replay_attn        one training-side call
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2604_18002_b200 import synth

CFG = dict(synth.CONFIGS[2])
WORKLOAD = "config2: 1.5B-shaped GQA rollout step (L28, 12q/2kv, d128, bf16, B64, 4096->2048 tokens, 256 decode steps)"
# the other workloads (--config 1, 3..7) are measurement aids; the default line is always config 2
OTHER_WORKLOADS = {
    1: "config1: tiny single-layer check (L1, 4q/4kv, d64, fp32, B4, 512 tokens of which 64 protected -> 256, 64 decode steps)",
    3: "config3: 7B-shaped ragged batch (L28, 28q/4kv, d128, bf16, B256, lengths 1024..8192 -> ceil(len/3), 128 decode steps)",
    4: "config4: per-(layer, KV head) eviction (L28, 12q/2kv, d128, bf16, B128, 16384 -> 8192 tokens, 7168 lists, 64 decode steps)",
    5: "config5: rollout loop (L28, 12q/2kv, d128, bf16, B64, 256 prompt + 8192 generated, a round every 512 tokens 768 -> 256, "
       "per-layer lists) + log-prob recompute of all 16 rounds",
    6: "config6: the paper's Countdown setting (L28, 12q/2kv, d128, bf16, B512 = 32 prompts x 16 rollouts, 256 prompt + 1024 generated, "
       "a round every 256 tokens 512 -> 256, units of 32 tokens, per-layer lists scored from K with 5 recent queries)",
    8: "config8: the paper's math setting with its own cadence (L28, 12q/2kv, d128, bf16, B2048, 337 prompt + 1050 generated, a round every "
       "350 tokens keeping 10 units of 32, per-layer lists scored from K, rounds at lengths with a short last unit: one cache length per "
       "(rollout, layer))",
    7: "config7: the paper's math setting (L28, 12q/2kv, d128, bf16, B2048 = 256 prompts x 8 rollouts, 352 prompt + 1056 generated, "
       "a round every 352 tokens 704 -> 352, units of 32 tokens, per-layer lists scored from K with 5 recent queries)",
}
METRIC = "evict+compact+decode tokens/sec at B=64"
W_RECENT = 5
# dram__bytes_read.sum + dram__bytes_write.sum over algorithmic K/V bytes for decode_stream_t_kernel, from the ncu
# capture summarised in profiles/decode_stream_t_kernel_config2.md (small case, scaled by tokens processed)
NCU_TRAFFIC_RATIO = 1.0118


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.idx), "-lms", "50"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples that arrived inside [t_begin, t_end] (the timed region)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, ln in self.lines:
            if t_begin is not None and not (t_begin <= ts <= t_end):
                continue
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def free_port():
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def spawn_ranks_if_needed(args):
    """`python bench.py --gpus N` with N > 1 outside a launcher: start N ranks of this script, one per GPU, and
    return their exit code (None when this process is itself a rank or N == 1)."""
    if args.gpus <= 1 or "RANK" in os.environ:
        return None
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    return subprocess.call(cmd, env=env)


def dist_setup(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world, device):
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def algorithmic_decode_bytes(cfg, visible_tokens_total):
    """K and V rows every decode launch must read: per (sequence, visible token) L*Hkv*2*d*2 bytes."""
    per_token = cfg["L"] * cfg["Hkv"] * 2 * cfg["d"] * 2
    return per_token * visible_tokens_total


# ------------------------------------------------------------------------------------ CUDA arm

def run_ngc(args):
    from paper_2604_18002_b200 import binding as ngc
    from paper_2604_18002_b200.rollout import HostStep, NgcRollout

    from paper_2604_18002_b200.sharding import list_base, shard_batch

    rank, world, local = dist_setup(args.gpus)
    if world != args.gpus and rank == 0:
        print(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s); reporting n_gpus = {world}", file=sys.stderr)
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    cfg = CFG
    L, Hq, Hkv, d, T, K, steps = cfg["L"], cfg["Hq"], cfg["Hkv"], cfg["d"], cfg["T"], cfg["budget"], cfg["steps"]
    if args.decode_steps:
        steps = args.decode_steps
    B_global = (args.batch or cfg["B"]) * world
    dtype = torch.bfloat16
    # weak scaling: the job's batch is world x 64 rollouts, cut into contiguous shards balanced by cached tokens
    # (all equal here); Philox streams use the global list index, so the draws do not depend on the sharding
    shard = shard_batch([T] * B_global, world)[rank]
    B = shard[1] - shard[0]
    seed = cfg["data_seed"] + 1000 * rank
    src = synth.make_cache(L, B, Hq, Hkv, d, dtype, [T] * B, capacity=T, seed=seed, outlier_channels=cfg["outliers"], device=dev)
    ro = NgcRollout(L, B, Hq, Hkv, d, dtype, capacity=T, n_max=T, k_max=K, lists=cfg["lists"], device=dev,
                    list_base=list_base(shard, 1), w=W_RECENT, kv=(src.k, src.v))
    del src
    lens0 = torch.full((B,), T, dtype=torch.int32, device=dev)
    logits = synth.make_logits(B, 1, T, seed=seed + 7, std=cfg["logit_std"], device=dev)
    n_t = lens0.clone()
    k_t = torch.full((B,), K, dtype=torch.int32, device=dev)
    q = synth.make_queries(L, B, Hq, d, dtype, seed=seed + 11, steps=steps, device=dev)
    nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=seed + 13, steps=steps, device=dev)
    q_recent = synth.normal((L, B, Hq, W_RECENT, d), seed + 17, dtype, device=dev)
    out = torch.empty((steps, L, B, Hq, d), dtype=torch.float32, device=dev)
    noise_seed = cfg["noise_seed"]

    ev_marks = []
    score_kernels = ngc.score_launches(ro.cache, W_RECENT)

    def one_step(step_idx, timed=False):
        """The whole hot path once.  Timed steps drop an event between the calls (score | sample | log-prob | compact |
        all decode calls of the step, none between those)."""
        marks = []

        def mark():
            if timed:
                e = torch.cuda.Event(enable_timing=True)
                e.record()
                marks.append(e)
        ro.cache.lens.copy_(lens0, non_blocking=True)
        mark()
        ngc.ngc_score_evict(ro.cache, q_recent, 1, cfg["lists"], ro.score_logits, ws=ro.ws_score, status=ro.status)
        mark()
        ngc.ngc_sample_evict(logits, n_t, None, k_t, noise_seed, step_idx, ro.kept_order, ro.kept_sorted, None,
                             list_base=ro.list_base, ws=ro.ws_sample, status=ro.status)
        mark()
        ngc.ngc_evict_logprob(logits, n_t, None, k_t, ro.kept_order, ro.logp, status=ro.status)
        mark()
        ngc.ngc_compact_kv(ro.cache, ro.kept_sorted, k_t, cfg["lists"], 1, status=ro.status)
        mark()
        ro.launches += score_kernels + 4          # score (group by group), sample 1, log-prob 1, compaction 2
        for s in range(steps):
            ro.decode_step(q[s], out[s], nk[s], nv[s])
        mark()
        if timed:
            ev_marks.append(marks)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()          # nvidia-smi takes a while to come up: start it before the warm-up
    for w in range(args.warmup):
        one_step(w)
    torch.cuda.synchronize()
    ro.check_status()

    launches0 = ro.launches
    barrier(world)
    torch.cuda.synchronize()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    wall0 = time.perf_counter()
    t0.record()
    for k in range(args.steps):
        one_step(args.warmup + k, timed=True)
    t1.record()
    torch.cuda.synchronize()
    wall1 = time.perf_counter()
    barrier(world)
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    ms_total = max_over_ranks(t0.elapsed_time(t1), world, dev)
    ro.check_status()
    launches = ro.launches - launches0
    ms_per_step = ms_total / args.steps
    tokens = B * steps * world
    value = tokens / (ms_per_step * 1e-3)

    # per-call times (median over the timed steps); roofline of the dominant kernel (decode): algorithmic K/V bytes
    # per launch / mean launch time; the same for compaction (every kept row read once and written once)
    call_names = ["score", "sample", "logprob", "compact", "decode"]
    per_call = {n: float(np.median([m[i].elapsed_time(m[i + 1]) for m in ev_marks])) for i, n in enumerate(call_names)}
    dec_ms = [m[4].elapsed_time(m[5]) for m in ev_marks]       # per step: all decode calls of the step
    mean_dec_ms = float(np.sum(dec_ms)) / (len(dec_ms) * steps)   # average duration of one decode call
    visible_total = sum(B * (K + s + 1) for s in range(steps)) / steps      # per launch, averaged over the step
    bytes_per_launch = algorithmic_decode_bytes(cfg, visible_total)
    peak, peak_kind = peaks()
    achieved = bytes_per_launch / (mean_dec_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "decode_stream_t_kernel (time per ngc_decode_attn_ragged call: attention with fused append + lens bump, launch gaps included)",
                "achieved": round(achieved, 1), "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": round(achieved / peak, 4),
                "traffic": int(args.traffic if args.traffic else NCU_TRAFFIC_RATIO * bytes_per_launch),
                "traffic_source": "ncu capture of a B=16 launch scaled by tokens processed (profiles/decode_stream_t_kernel_config2.md)", "bytes_per_launch": int(bytes_per_launch),
                "ms_per_launch": round(mean_dec_ms, 4), "decode_share_of_step": round(sum(dec_ms) / ms_total, 4),
                "frac_of_nominal_8TBs": round(achieved / 8000.0, 4)}
    row_bytes = L * Hkv * 2 * d * 2
    compact_bytes = 2.0 * B * K * row_bytes
    cmp_gbs = compact_bytes / (per_call["compact"] * 1e-3) / 1e9
    compact = {"kernel": "compact_kernel<16> (+ the length kernel behind it: time per ngc_compact_kv call)", "bytes": int(compact_bytes),
               "ms": round(per_call["compact"], 4), "GB/s": round(cmp_gbs, 1), "frac": round(cmp_gbs / peak, 4), "peak_kind": f"of {peak_kind}",
               "frac_of_nominal_8TBs": round(cmp_gbs / 8000.0, 4),
               "note": "algorithmic bytes = every kept row of K and V read once and written once (2 x B x kept x 28672 B)"}

    result = {"metric": METRIC, "value": round(value, 1), "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
              "warmup": args.warmup, "ms_per_step": round(ms_per_step, 3), "higher_is_better": True, "scaling": "weak",
              "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
              "config": {"workload": WORKLOAD, "decode_steps": steps, "batch_per_gpu": B, "batch_global": B_global,
                         "parallelism": f"batch-shard x{world} (contiguous shards of {B}, global Philox list ids), no collective",
                         "l2": "inputs larger than L2 (7.5 GB cache streamed per decode step)", "score_in_step": True,
                         "logits": "synthetic N(0, var 2), shared list"},
              "gpu_launches": int(launches), "roofline": roofline, "compact": compact,
              "per_call_ms": {n: round(v, 4) for n, v in per_call.items()}}
    if clocks is not None:
        result["clocks"] = clocks

    # ---- end to end from pinned host buffers (all ranks take part, rank 0 reports) ----
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        hs = HostStep(ro, steps, double_buffer=True)      # next step's cache uploads while this step computes
        pin = dict(pin_memory=True)
        h_k = torch.empty(ro.cache.k.shape, dtype=dtype, **pin).copy_(ro.cache.k)
        h_v = torch.empty(ro.cache.v.shape, dtype=dtype, **pin).copy_(ro.cache.v)
        h_lens = torch.empty(B, dtype=torch.int32, **pin).copy_(lens0)
        h_logits = torch.empty(logits.shape, dtype=torch.float32, **pin).copy_(logits)
        h_q = torch.empty(q.shape, dtype=dtype, **pin).copy_(q)
        h_nk = torch.empty(nk.shape, dtype=dtype, **pin).copy_(nk)
        h_nv = torch.empty(nv.shape, dtype=dtype, **pin).copy_(nv)
        h_qr = torch.empty(q_recent.shape, dtype=dtype, **pin).copy_(q_recent)
        h_out = torch.empty(out.shape, dtype=torch.float32, **pin)
        h_ko = torch.empty(ro.kept_order.shape, dtype=torch.int32, **pin)
        h_lp = torch.empty(ro.logp.shape, dtype=torch.float64, **pin)
        torch.cuda.synchronize()

        def host_step(i):
            return hs.run(h_k, h_v, h_lens, h_logits, h_q, h_nk, h_nv, h_out, h_ko, h_lp, n_t, None, k_t, noise_seed, i,
                          h_q_recent=h_qr, d_q_recent=q_recent, prefetch_next=(h_k, h_v))
        host_step(0)
        torch.cuda.synchronize()
        barrier(world)
        c0 = time.perf_counter()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(e2e_steps):
            h2d, d2h = host_step(100 + i)
        e1.record()
        torch.cuda.synchronize()
        wall = time.perf_counter() - c0
        barrier(world)
        e2e_ms = max_over_ranks(max(e0.elapsed_time(e1), wall * 1e3), world, dev) / e2e_steps
        ro.check_status()
        result["e2e"] = {"value": round(tokens / (e2e_ms * 1e-3), 1), "unit": "tokens/s", "h2d_bytes_per_step": int(h2d),
                         "d2h_bytes_per_step": int(d2h), "ms_per_step": round(e2e_ms, 3), "steps": e2e_steps,
                         "api": "paper_2604_18002_b200.rollout.HostStep.run (pinned host buffers; every step uploads the next step's cache into a second device buffer while it computes, decode inputs and outputs stream on copy streams)"}
        del h_k, h_v, h_q, h_nk, h_nv, h_out, hs

    # ---- the 7B-shaped ragged batch, per call (one GPU only): same kernels, second target shape ----
    if world == 1 and not args.no_config3:
        del ro, q, nk, nv, out, logits, q_recent
        torch.cuda.empty_cache()
        sub = argparse.Namespace(**vars(args))
        sub.config, sub.steps, sub.warmup, sub.batch, sub.decode_steps, sub.graph, sub.paged = 3, args.config3_steps, 3, 0, 0, False, False
        free, _ = torch.cuda.mem_get_info()
        if free < 90 * 2 ** 30:
            result["config3"] = {"skipped": f"needs 90 GB of free device memory, {free / 2 ** 30:.0f} GB available"}
        else:
            r3 = measure_other(sub)
            result["config3"] = {k: r3[k] for k in ("value", "unit", "ms_per_step", "steps", "warmup", "per_call_ms", "roofline", "compact",
                                                   "gpu_launches", "clocks")}
            result["config3"]["workload"] = r3["config"]["workload"]
            torch.cuda.empty_cache()

    # ---- CPU oracle on a bounded sample (rank 0, N = 1 only) ----
    if rank == 0 and world == 1 and not args.no_cpu:
        result["cpu_baseline"] = cpu_baseline_sample(args.cpu_seqs, args.cpu_decode_steps)
    if rank == 0:
        print(json.dumps(result), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------ other workloads (measurement aid)

def run_other(args):
    print(json.dumps(measure_other(args)), flush=True)


def measure_other(args):
    """Configs 1 and 3..8 on one GPU: the same hot path, timed per phase.  Decode inputs come from a ring of
    `ring` distinct steps (the full set would not fit beside the 60+ GB caches); outputs of a step overwrite the ring slot."""
    from paper_2604_18002_b200 import binding as ngc
    from paper_2604_18002_b200.rollout import NgcRollout

    torch.cuda.set_device(0)
    dev = "cuda:0"
    cid = args.config
    cfg = synth.CONFIGS[cid]
    L, B, Hq, Hkv, d, steps = cfg["L"], args.batch or cfg["B"], cfg["Hq"], cfg["Hkv"], cfg["d"], args.decode_steps or cfg["steps"]
    dtype = torch.float32 if cfg["dtype"] == "f32" else torch.bfloat16
    lists = cfg["lists"]
    loop = cid >= 5                      # grow-then-evict loop (rounds) instead of one round + decode
    block = cfg.get("block", 1)
    from_score = cid >= 6               # the draw uses the scores of the real K, not synthetic logits
    if loop:
        prompt, cadence, K = cfg["T"], cfg["cadence"], cfg["budget"]
        rounds = max(1, steps // cadence)
        steps = rounds * cadence
        lens = torch.full((B,), prompt, dtype=torch.int32)
        budget = torch.full((B,), K, dtype=torch.int32)              # in units
        cap = torch.full((B,), prompt + cadence + block, dtype=torch.int64)
        n_evict = torch.full((B,), (prompt + cadence + block - 1) // block, dtype=torch.int32)
    else:
        if isinstance(cfg["T"], tuple):
            lens = synth.ragged_lens(B, cfg["T"][0], cfg["T"][1], cfg["len_seed"])
        else:
            lens = torch.full((B,), cfg["T"], dtype=torch.int32)
        budget = torch.ceil(lens.double() / 3).to(torch.int32) if cfg["budget"] == "third" else torch.full((B,), cfg["budget"], dtype=torch.int32)
        cap = torch.maximum(lens.long(), budget.long() + steps)
        n_evict = lens
    n_max, k_max = max(int(n_evict.max()), (int(cap.max()) + block - 1) // block), int(budget.max())
    src = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=cap, seed=cfg["data_seed"], outlier_channels=cfg["outliers"], device=dev)
    per_list = bool(cfg.get("per_list_lens"))
    ro = NgcRollout(L, B, Hq, Hkv, d, dtype, capacity=cap, n_max=n_max, k_max=k_max, lists=lists, block=block, device=dev, w=W_RECENT,
                    kv=(src.k, src.v), per_list_lens=per_list)
    del src
    G = ro.G
    lens0 = lens.to(dev)
    if per_list:
        lens0 = lens0[:, None].repeat(1, G).contiguous()
    logits = ro.score_logits if from_score else synth.make_logits(B, G, n_max, seed=cfg["data_seed"] + 7, std=cfg["logit_std"], device=dev)
    n_t, k_t = n_evict.to(dev), budget.to(dev)
    p_t = torch.full((B,), cfg["n_protect"], dtype=torch.int32, device=dev) if cfg["n_protect"] else None
    ring = ((cadence if loop else steps) if args.graph else min(steps, args.ring))
    q = synth.make_queries(L, B, Hq, d, dtype, seed=11, steps=ring, device=dev)
    nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=13, steps=ring, device=dev)
    q_recent = synth.normal((L, B, Hq, W_RECENT, d), 17, dtype, device=dev)
    out = torch.empty((ring, L, B, Hq, d), dtype=torch.float32, device=dev)
    row_bytes = L * Hkv * 2 * d * (4 if dtype == torch.float32 else 2)
    names = ["score", "sample", "logprob", "compact", "decode", "recompute"]
    acc = {n: [] for n in names}

    paged = None
    if args.paged:
        # same memory viewed as page pools (one eviction unit = one page): eviction edits the tables only
        assert loop and block in (32, 64), "--paged needs a block-eviction workload (--config 6 or 7)"
        pages_cap = (prompt + cadence + block) // block
        table = torch.arange(pages_cap, dtype=torch.int32, device=dev).repeat(B, G, 1).contiguous()
        table0 = table.clone()
        paged = ngc.NgcPagedCache(ro.cache.k.view(L, Hkv, B * pages_cap, block, d), ro.cache.v.view(L, Hkv, B * pages_cap, block, d),
                                  table, ro.cache.lens, Hq, lists)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    score_kernels = ngc.score_launches(ro.cache, W_RECENT)

    def eviction(rnd, t):
        e = [ev() for _ in range(5)]
        e[0].record()
        # with a length per list the scoring call itself reports the units of each rollout's longest layer (n_t) and
        # writes -inf into the units a shorter layer lacks
        if paged is not None:
            ngc.ngc_score_evict_paged(paged, q_recent, ro.score_logits, ws=ro.ws_score, status=ro.status)
        else:
            ngc.ngc_score_evict(ro.cache, q_recent, ro.block, lists, ro.score_logits, ws=ro.ws_score, status=ro.status,
                                n_units_out=n_t if per_list else None)
        e[1].record()
        ngc.ngc_sample_evict(logits, n_t, p_t, k_t, cfg["noise_seed"], rnd, ro.kept_order, ro.kept_sorted, None, ws=ro.ws_sample, status=ro.status)
        e[2].record()
        ngc.ngc_evict_logprob(logits, n_t, p_t, k_t, ro.kept_order, ro.logp, status=ro.status)
        e[3].record()
        if paged is not None:
            ngc.ngc_evict_pages(paged, ro.kept_sorted, k_t, status=ro.status)
        else:
            ngc.ngc_compact_kv(ro.cache, ro.kept_sorted, k_t, lists, block, status=ro.status)
        e[4].record()
        ro.launches += score_kernels + 4 + (1 if G > 1 and not per_list and paged is None else 0)   # score, sample 1, log-prob 1, compaction 2 (+ check)
        t.append(e)

    graph = None

    def decode(n, t):
        e0, e1 = ev(), ev()
        e0.record()
        if graph is not None:
            graph.replay()          # all decode steps of the round with one launch from the host
            ro.launches += 2 * n
            e1.record()
            t.append((e0, e1))
            return
        for s in range(n):
            if paged is not None:
                ngc.ngc_decode_attn_paged(paged, q[s % ring], out[s % ring], nk[s % ring], nv[s % ring], ws=ro.ws_decode, status=ro.status)
                ro.launches += 2
            else:
                ro.decode_step(q[s % ring], out[s % ring], nk[s % ring], nv[s % ring])
        e1.record()
        t.append((e0, e1))

    if loop:
        all_logits = logits.unsqueeze(0).expand(rounds, B, G, n_max).contiguous()
        all_ko = torch.zeros((rounds, B, G, k_max), dtype=torch.int32, device=dev)
        all_lp = torch.empty((rounds, B, G), dtype=torch.float64, device=dev)
        n_all, k_all = n_t.unsqueeze(0).expand(rounds, B).contiguous(), k_t.unsqueeze(0).expand(rounds, B).contiguous()

    def one_step(i, rec):
        ro.cache.lens.copy_(lens0, non_blocking=True)
        if paged is not None:
            paged.page_table.copy_(table0, non_blocking=True)
        ev_t, dec_t, rc = [], [], None
        if loop:
            for r in range(rounds):
                decode(cadence, dec_t)
                eviction(i * rounds + r, ev_t)
                all_ko[r].copy_(ro.kept_order, non_blocking=True)
                if from_score:
                    all_logits[r].copy_(logits, non_blocking=True)
            rc = (ev(), ev())
            rc[0].record()
            ngc.ngc_evict_logprob(all_logits, n_all, None, k_all, all_ko, all_lp, status=ro.status)
            rc[1].record()
            ro.launches += 1
        else:
            eviction(i, ev_t)
            decode(steps, dec_t)
        rec.append((ev_t, dec_t, rc))

    sampler = ClockSampler(0)
    sampler.start()
    for w in range(args.warmup):
        one_step(w, [])
    torch.cuda.synchronize()
    ro.check_status()
    if args.graph:
        assert paged is None, "--graph and --paged are separate measurements"
        graph = ro.capture_decode_steps(q[: (cadence if loop else steps)], out, nk, nv)
        one_step(args.warmup, [])
        torch.cuda.synchronize()
    rec = []
    launches0 = ro.launches
    t0, t1 = ev(), ev()
    wall0 = time.perf_counter()
    t0.record()
    for k in range(args.steps):
        one_step(args.warmup + k, rec)
    t1.record()
    torch.cuda.synchronize()
    wall1 = time.perf_counter()
    clocks = sampler.stop(wall0, wall1)
    ro.check_status()
    ms_per_step = t0.elapsed_time(t1) / args.steps
    for ev_t, dec_t, rc in rec:
        for e in ev_t:
            for i, n in enumerate(names[:4]):
                acc[n].append(e[i].elapsed_time(e[i + 1]))
        acc["decode"].append(sum(a.elapsed_time(b) for a, b in dec_t))
        if rc:
            acc["recompute"].append(rc[0].elapsed_time(rc[1]))
    tokens = B * steps
    # algorithmic K/V bytes: every visible token of every decode launch; every kept row read + written by compaction
    kept = float(budget.sum())
    if loop:
        kept *= block
        # after the first round the cache restarts from the kept units (a short last unit can cost up to block - 1 tokens less)
        vis = B * (sum(prompt + s + 1 for s in range(cadence)) + (rounds - 1) * sum(K * block + s + 1 for s in range(cadence)))
        score_bytes = float(n_evict.sum()) * block * row_bytes / 2
    else:
        vis = sum(kept + B * (s + 1) for s in range(steps))
        score_bytes = float(lens.sum()) * row_bytes / 2
    compact_bytes = 2 * kept * row_bytes
    dec_ms = float(np.mean(acc["decode"]))
    peak, peak_kind = peaks()
    med = {n: round(float(np.median(v)), 4) for n, v in acc.items() if v}
    dec_gbs = vis * row_bytes / (dec_ms * 1e-3) / 1e9
    cmp_gbs = compact_bytes / (med["compact"] * 1e-3) / 1e9
    result = {"metric": "evict+compact+decode tokens/sec", "value": round(tokens / (ms_per_step * 1e-3), 1), "unit": "tokens/s", "n_gpus": 1,
              "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_per_step, 3), "dtype": cfg["dtype"], "data": "synthetic",
              "config": {"workload": OTHER_WORKLOADS[cid], "batch": B, "decode_steps": steps, "input_ring": ring,
                         "layout": "paged (eviction edits page tables, no K/V movement)" if paged is not None else "contiguous strips, in-place compaction",
                         "decode_loop": "one CUDA graph per round" if args.graph else "eager launches"},
              "per_call_ms": med,
              "roofline": {"bound": "hbm", "kernel": "decode_stream_t_kernel (all decode calls of a step, launch gaps included)",
                           "achieved": round(dec_gbs, 1), "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                           "frac": round(dec_gbs / peak, 4), "frac_of_nominal_8TBs": round(dec_gbs / 8000.0, 4),
                           "decode_ms_per_step": round(dec_ms, 3), "decode_calls": steps, "traffic": None},
              "compact": {"bytes": int(compact_bytes), "ms": med["compact"], "GB/s": round(cmp_gbs, 1), "frac": round(cmp_gbs / peak, 4),
                          "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": round(cmp_gbs / 8000.0, 4),
                          "note": "algorithmic bytes = every kept row read once and written once (rows already in place are skipped by the kernel)"},
              "score": {"bytes": int(score_bytes), "GB/s": round(score_bytes / (med["score"] * 1e-3) / 1e9, 1),
                        "note": "algorithmic bytes = K read once; the kernel streams K twice"},
              "gpu_launches": int(ro.launches - launches0), "clocks": clocks}
    return result


# ------------------------------------------------------------------------------------ training-side kernels (measurement aid)

def run_kernel(args):
    """Times one training-side call on one GPU: `--kernel score_backward` (gradient of the eviction scores at
    the config-2 shape) or `--kernel replay_attn` (replay attention over the rollout-loop history of config 5,
    `--layers` of its 28 layers)."""
    from paper_2604_18002_b200 import binding as ngc
    torch.cuda.set_device(0)
    dev = "cuda:0"
    peak_hbm, peak_kind = peaks()
    st = ngc.new_status(dev)

    def best_of(fn, reps):
        best = 1e9
        for rep in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if rep:
                best = min(best, e0.elapsed_time(e1))
        return best

    if args.kernel == "score_backward":
        cfg = synth.CONFIGS[2]
        L, Hq, Hkv, d, T, B = cfg["L"], cfg["Hq"], cfg["Hkv"], cfg["d"], cfg["T"], args.batch or cfg["B"]
        c = synth.make_cache(L, B, Hq, Hkv, d, torch.bfloat16, [T] * B, capacity=T, seed=0, device=dev)
        dc = ngc.NgcCache(c.k, c.v, c.seq_off, c.lens, Hq, T)
        qr = synth.normal((L, B, Hq, W_RECENT, d), 1, torch.bfloat16, device=dev)
        up = synth.make_logits(B, 1, T, seed=2, device=dev)
        gq = torch.empty(qr.shape, dtype=torch.float32, device=dev)
        gk = torch.empty_like(c.k)
        ws = ngc.alloc_workspace(ngc.workspace_bytes(ngc.OP_SCORE_BACKWARD, dc), dev)
        ms = best_of(lambda: ngc.ngc_score_evict_backward(dc, qr, 1, ngc.LISTS_SHARED, up, gq, gk, ws=ws, status=st), args.steps)
        nbytes = 3 * L * Hkv * B * T * d * 2
        res = {"kernel": "ngc_score_evict_backward", "workload": f"config-2 shape, B={B}, T={T}, w={W_RECENT}, shared list", "ms": round(ms, 3),
               "roofline": {"bound": "hbm", "achieved": round(nbytes / ms / 1e6, 1), "peak": peak_hbm, "peak_kind": f"of {peak_kind}",
                            "unit": "GB/s", "frac": round(nbytes / ms / 1e6 / peak_hbm, 4), "bytes": "K read twice + dK written once"}}
    else:
        cfg = synth.CONFIGS[5]
        L, Hq, Hkv, d, B = args.layers, cfg["Hq"], cfg["Hkv"], cfg["d"], args.batch or cfg["B"]
        K, delta, prompt = cfg["budget"], cfg["cadence"], cfg["T"]
        R, alive = cfg["steps"] // delta, prompt + delta
        T = prompt + R * delta
        g = torch.Generator(device=dev)
        g.manual_seed(0)
        u = torch.rand((R, B, L, alive), device=dev, generator=g)
        ks = torch.sort(torch.topk(u, K, dim=-1).indices, dim=-1).values.to(torch.int32).contiguous()
        del u
        budget = torch.full((R, B), K, dtype=torch.int32, device=dev)
        alive_before = torch.full((R, B), alive, dtype=torch.int32, device=dev)
        total_before = (alive + delta * torch.arange(R, device=dev, dtype=torch.int32))[:, None].repeat(1, B).contiguous()
        pos = torch.empty((R, B, L, K), dtype=torch.int32, device=dev)
        cnt = torch.empty((R, B, L), dtype=torch.int32, device=dev)
        ngc.ngc_replay_visibility(ks, budget, alive_before, total_before, 1, alive, pos, cnt, status=st)
        c = synth.make_cache(L, B, Hq, Hkv, d, torch.bfloat16, [T] * B, capacity=T, seed=0, device=dev)
        dc = ngc.NgcCache(c.k, c.v, c.seq_off, c.lens, Hq, T)
        q = synth.normal((L, B, Hq, T, d), 1, torch.bfloat16, device=dev)
        out = torch.empty((L, B, Hq, T, d), dtype=torch.bfloat16, device=dev)
        ms = best_of(lambda: ngc.ngc_replay_attn(dc, q, out, pos, cnt, total_before, lists=ngc.LISTS_PER_LAYER, status=st,
                                                 variant=args.variant), args.steps)
        vis = sum(t + 1 for t in range(alive)) + sum(sum(K + s + 1 for s in range(min(delta, T - (alive + (r - 1) * delta)))) for r in range(1, R + 1))
        flops = 4.0 * d * vis * Hq * L * B
        tf_peak = 1590.0
        pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(pk):
            with open(pk) as f:
                tf_peak = float(json.load(f)["bf16_tflops"])
        res = {"kernel": "ngc_replay_attn", "path": {None: "default (tcgen05)", 0: "default (tcgen05)", 1: "mma.sync", 2: "tcgen05"}[args.variant],
               "workload": f"config-5 history: {L} layers, B={B}, T={T}, {R} rounds, {K} kept per round and layer",
               "ms": round(ms, 3),
               "roofline": {"bound": "tensor", "achieved": round(flops / ms / 1e9, 1), "peak": tf_peak, "unit": "TFLOP/s",
                            "frac": round(flops / ms / 1e9 / tf_peak, 4), "flops": "4*d per visible key per query per head (masked keys not counted)"}}
    torch.cuda.synchronize()
    res["dev_status"] = int(st.item())
    print(json.dumps(res), flush=True)


# ------------------------------------------------------------------------------------ CPU oracle arm

def oracle_step(cache_np, logits, q, nk, nv, qr, K, rnd, decode_steps, seed):
    """One step of the workload through the CPU oracle, as it stands."""
    import oracle
    k, v, so, lens = cache_np
    B = lens.shape[0]
    budget = np.full(B, K, np.int32)
    oracle.score_evict(k, so, lens, qr, 1, 0)
    ko, ks, _, st = oracle.sample_evict(logits, lens, None, budget, K, seed=seed, rnd=rnd)
    oracle.evict_logprob(logits, lens, None, budget, ko)
    kc, vc, nl, rc = oracle.compact_kv(k, v, so, lens, ks, budget, 0)
    lens2 = nl.copy()
    for s in range(decode_steps):
        oracle.decode_attn(kc, vc, so, lens2, q[s], nk[s], nv[s])


def make_cpu_sample(n_seqs, decode_steps):
    cfg = CFG
    L, Hq, Hkv, d, T = cfg["L"], cfg["Hq"], cfg["Hkv"], cfg["d"], cfg["T"]
    c = synth.make_cache(L, n_seqs, Hq, Hkv, d, torch.bfloat16, [T] * n_seqs, capacity=T, seed=0, outlier_channels=cfg["outliers"])
    logits = synth.make_logits(n_seqs, 1, T, seed=7, std=cfg["logit_std"]).numpy()
    q = synth.to_numpy(synth.make_queries(L, n_seqs, Hq, d, torch.bfloat16, seed=11, steps=decode_steps))
    nk, nv = synth.make_new_kv(L, n_seqs, Hkv, d, torch.bfloat16, seed=13, steps=decode_steps)
    qr = synth.to_numpy(synth.normal((L, n_seqs, Hq, W_RECENT, d), 17, torch.bfloat16))
    cache_np = (synth.to_numpy(c.k), synth.to_numpy(c.v), c.seq_off.numpy(), c.lens.numpy())
    return cache_np, logits, q, synth.to_numpy(nk), synth.to_numpy(nv), qr


def cpu_baseline_sample(n_seqs, decode_steps):
    import oracle
    data = make_cpu_sample(n_seqs, decode_steps)
    t0 = time.perf_counter()
    oracle_step(*data, CFG["budget"], 0, decode_steps, CFG["noise_seed"])
    dt = time.perf_counter() - t0
    return {"value": round(n_seqs * decode_steps / dt, 2), "unit": "tokens/s", "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{n_seqs} of {CFG['B']} sequences, one eviction round (score+sample+logprob+compact) + {decode_steps} of "
                      f"{CFG['steps']} decode steps, {dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    if "LOCAL_RANK" in os.environ and oracle.threads() == 1:
        # the multi-rank launcher pins OpenMP to one thread per rank; this arm runs on rank 0 alone, on the host's cores
        import ctypes
        try:
            ctypes.CDLL("libgomp.so.1").omp_set_num_threads(len(os.sched_getaffinity(0)))
        except OSError:
            pass
    n_seqs, dsteps = args.cpu_seqs, args.cpu_decode_steps
    data = make_cpu_sample(n_seqs, dsteps)
    for w in range(args.warmup):
        oracle_step(*data, CFG["budget"], w, dsteps, CFG["noise_seed"])
    t0 = time.perf_counter()
    for k in range(args.steps):
        oracle_step(*data, CFG["budget"], args.warmup + k, dsteps, CFG["noise_seed"])
    dt = (time.perf_counter() - t0) / args.steps
    value = n_seqs * dsteps / dt
    sample = (f"each step: {n_seqs} of {CFG['B']} sequences, one eviction round + {dsteps} of {CFG['steps']} decode steps "
              f"({dt:.1f} s per step)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 2), "unit": "tokens/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 1), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": round(value, 2), "unit": "tokens/s", "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 2), "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def run_launch_check(args):
    """Plumbing check of the multi-rank launch (no GPU work): every rank joins the process group (gloo without CUDA),
    takes its shard of the job's batch, meets the barrier and the max-over-ranks reduction the timed region uses;
    rank 0 prints what it saw."""
    from paper_2604_18002_b200.sharding import shard_batch
    rank, world, local = dist_setup(args.gpus)
    lens = synth.ragged_lens(64 * world, 1024, 8192, 2).tolist()
    shards = shard_batch(lens, world)
    barrier(world)
    dev = f"cuda:{local}" if torch.cuda.is_available() else "cpu"
    top = max_over_ranks(float(rank + 1), world, dev)
    if rank == 0:
        print(json.dumps({"impl": "launch-check", "n_gpus": world, "requested": args.gpus, "max_over_ranks": top,
                          "shards": shards, "shard_tokens": [sum(lens[a:b]) for a, b in shards]}), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ngc", choices=["ngc", "reference", "launch-check"],
                    help="ngc = the CUDA library; reference = the CPU oracle on a bounded sample; launch-check = rank plumbing only")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's 256 decode steps (profiling only)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's B = 64 (profiling only)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-config3", action="store_true", help="skip the per-call pass over the 7B-shaped ragged batch")
    ap.add_argument("--config3-steps", type=int, default=2)
    ap.add_argument("--cpu-seqs", type=int, default=4)
    ap.add_argument("--cpu-decode-steps", type=int, default=48)
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5, 6, 7, 8],
                    help="2 = the benchmark workload (default); 1, 3..7 = the other workloads, one GPU, per-phase timing only")
    ap.add_argument("--kernel", default=None, choices=["score_backward", "replay_attn"],
                    help="time one training-side call instead of the benchmark step (one GPU)")
    ap.add_argument("--layers", type=int, default=4, help="--kernel replay_attn: layers of the history to run")
    ap.add_argument("--variant", type=int, default=None, choices=[0, 1, 2],
                    help="--kernel replay_attn: device path (1 = the warp-level MMA kernel, 2 = tcgen05; default: what the library picks)")
    ap.add_argument("--graph", action="store_true", help="--config 1|3..7: replay the decode calls of a round as one CUDA graph")
    ap.add_argument("--paged", action="store_true", help="--config 6|7 only: paged cache, one eviction unit = one page")
    ap.add_argument("--ring", type=int, default=8, help="distinct decode-input steps kept on the device for --config 3|4|5")
    ap.add_argument("--traffic", type=float, default=None, help="dram bytes per decode launch from an ncu capture (profiles/)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ngc" and not (args.decode_steps or args.batch):
        args.warmup = 3
    rc = spawn_ranks_if_needed(args)
    if rc is not None:
        raise SystemExit(rc)
    if args.impl == "reference":
        run_reference(args)
    elif args.impl == "launch-check":
        run_launch_check(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the CPU oracle")
        if args.kernel:
            run_kernel(args)
        elif args.config != 2:
            run_other(args)
        else:
            run_ngc(args)


if __name__ == "__main__":
    main()
