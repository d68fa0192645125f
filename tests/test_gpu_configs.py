"""The five workload configurations at full size on the GPU, checked against
the CPU oracle: kept sets, orders and compacted rows bit-exact; log-probs
<= 1e-3 abs; attention <= 1e-5 abs (fp32) / <= 2e-2 relative (bf16).

Inputs are generated on the GPU (seeded) in the same launch configuration the
benchmark uses; what the oracle needs (logits, the strips of a few sampled
sequences, their queries and new rows) is copied back to the host, so both
sides see the same bytes.  Integer outputs are checked for EVERY list.  The
1.5B- and the 7B-shaped configurations check cache rows and attention for
EVERY sequence (whole layers streamed through host memory, attention at the
first, a middle and the last decode step); the others for sampled sequences.  Eq. (1) is checked literally on sampled lists and through the
(cross-checked) scan for all of them.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import max_rel_err_per_vector, ngc
from paper_2604_18002_b200 import synth

pytestmark = pytest.mark.gpu


def need_gpu_gb(gb):
    free, total = torch.cuda.mem_get_info()
    if free < gb * 2 ** 30:
        pytest.skip(f"needs {gb} GB of free device memory, {free / 2 ** 30:.0f} GB available")


class SampledSeqs:
    """Host mirror of a few sequences of a device cache: their strips packed as a small cache."""

    def __init__(self, cache, seqs, cap):
        self.seqs = list(seqs)
        L, Hkv, R, d = cache.k.shape
        so = cache.seq_off.cpu().numpy()
        n = len(self.seqs)
        self.so = np.arange(n + 1, dtype=np.int64) * cap
        dt = np.uint16 if cache.k.dtype == torch.bfloat16 else np.float32
        self.k = np.zeros((L, Hkv, n * cap, d), dt)
        self.v = np.zeros((L, Hkv, n * cap, d), dt)
        self.src_off = so
        self.cap = cap
        self.pull(cache)

    def pull(self, cache):
        for i, b in enumerate(self.seqs):
            o = int(self.src_off[b])
            c = min(self.cap, int(self.src_off[b + 1]) - o)
            self.k[:, :, i * self.cap:i * self.cap + c] = synth.to_numpy(cache.k[:, :, o:o + c])
            self.v[:, :, i * self.cap:i * self.cap + c] = synth.to_numpy(cache.v[:, :, o:o + c])


def check_attention(got, ref, dtype):
    if dtype == torch.float32:
        assert np.max(np.abs(got - ref)) <= 1e-5
    else:
        assert max_rel_err_per_vector(got, ref) <= 2e-2


def run_round_and_decode(cfg_id, B=None, steps=None, check_steps=None, seqs=(0, 1), literal_lists=8, use_score=False):
    """One eviction round + decode steps of configs 1-4 at full size; returns nothing, asserts parity."""
    b = ngc()
    from paper_2604_18002_b200.rollout import NgcRollout
    cfg = synth.CONFIGS[cfg_id]
    L, Hq, Hkv, d = cfg["L"], cfg["Hq"], cfg["Hkv"], cfg["d"]
    B = B or cfg["B"]
    steps = steps or cfg["steps"]
    dtype = torch.float32 if cfg["dtype"] == "f32" else torch.bfloat16
    dev = "cuda"
    if isinstance(cfg["T"], tuple):
        lens = synth.ragged_lens(B, cfg["T"][0], cfg["T"][1], cfg["len_seed"])
    else:
        lens = torch.full((B,), cfg["T"], dtype=torch.int32)
    if cfg["budget"] == "third":
        budget = torch.ceil(lens.double() / 3).to(torch.int32)
    else:
        budget = torch.full((B,), cfg["budget"], dtype=torch.int32)
    cap = torch.maximum(lens.long(), budget.long() + steps)
    n_max, k_max = int(lens.max()), int(budget.max())
    lists = cfg["lists"]
    src = synth.make_cache(L, B, Hq, Hkv, d, dtype, lens, capacity=cap, seed=cfg["data_seed"],
                           outlier_channels=cfg["outliers"], device=dev)
    ro = NgcRollout(L, B, Hq, Hkv, d, dtype, capacity=cap, n_max=n_max, k_max=k_max, lists=lists, device=dev,
                    with_score=use_score, kv=(src.k, src.v))
    ro.cache.lens.copy_(src.lens)
    del src
    G = ro.G
    logits = synth.make_logits(B, G, n_max, seed=cfg["data_seed"] + 7, std=cfg["logit_std"], device=dev)
    n_t = lens.to(dev)
    p_np = np.full(B, cfg["n_protect"], np.int32)
    p_t = torch.as_tensor(p_np).to(dev) if cfg["n_protect"] else None
    k_t = budget.to(dev)
    seqs = [s for s in seqs if s < B]
    host_cap = int(cap.max())
    mirror = SampledSeqs(ro.cache, seqs, host_cap)            # strips before eviction

    # ---- eviction round on the GPU
    ro.eviction_round(n_t, p_t, k_t, cfg["noise_seed"], 0, logits=logits)
    torch.cuda.synchronize()
    ro.check_status()

    # ---- sample: every list, bit-exact
    lg = logits.cpu().numpy()
    lens_np, budget_np = lens.numpy(), budget.numpy()
    r_ko, r_ks, _, r_st = oracle.sample_evict(lg, lens_np, p_np, budget_np, k_max, seed=cfg["noise_seed"], rnd=0)
    assert not r_st.any()
    assert np.array_equal(ro.kept_order.cpu().numpy(), r_ko), "kept_order differs"
    assert np.array_equal(ro.kept_sorted.cpu().numpy(), r_ks), "kept_sorted differs"
    # invariants that hold at any size
    assert np.all((r_ks >= 0).sum(-1) == budget_np[:, None])

    # ---- log-prob: scan for all lists, Eq. (1) literally for a few
    got_lp = ro.logp.cpu().numpy()
    ref_scan, rc = oracle.evict_logprob_scan(lg, lens_np, p_np, budget_np, r_ko)
    assert rc == 0 and np.max(np.abs(got_lp - ref_scan)) <= 1e-3
    pick = np.unique(np.linspace(0, B * G - 1, min(literal_lists, B * G)).astype(int))
    pb, pg = pick // G, pick % G
    ref_lit, rc = oracle.evict_logprob(lg[pb, pg][:, None], lens_np[pb], p_np[pb], budget_np[pb], r_ko[pb, pg][:, None])
    assert rc == 0 and np.max(np.abs(got_lp[0, pb, pg] - ref_lit[0, :, 0])) <= 1e-3

    # ---- compaction: sampled sequences, bit-exact on the live rows
    sel = np.array(seqs)
    kc, vc, nl, rc = oracle.compact_kv(mirror.k, mirror.v, mirror.so, lens_np[sel], r_ks[sel], budget_np[sel], lists)
    assert rc == 0
    new_lens = ro.cache.lens.cpu().numpy()
    assert np.array_equal(new_lens, budget_np)
    after = SampledSeqs(ro.cache, seqs, host_cap)
    for i in range(len(seqs)):
        sl = slice(i * host_cap, i * host_cap + int(nl[i]))
        assert np.array_equal(after.k[:, :, sl], kc[:, :, sl]) and np.array_equal(after.v[:, :, sl], vc[:, :, sl])

    # ---- decode steps: GPU runs every step on the whole batch; the oracle follows the sampled sequences
    check_steps = sorted(set(check_steps if check_steps is not None else [0, steps // 2, steps - 1]))
    o_lens = nl.copy()
    out = torch.empty((L, B, Hq, d), dtype=torch.float32, device=dev)
    for s in range(steps):
        q = synth.make_queries(L, B, Hq, d, dtype, seed=1000 + s, device=dev)
        nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=5000 + 2 * s, device=dev)
        ro.decode_step(q, out, nk, nv)
        nk_h = synth.to_numpy(nk[:, seqs])
        nv_h = synth.to_numpy(nv[:, seqs])
        if s in check_steps:
            ref, rc = oracle.decode_attn(kc, vc, mirror.so, o_lens, synth.to_numpy(q[:, seqs]), nk_h, nv_h)
            assert rc == 0
            got = out[:, seqs].cpu().numpy().astype(np.float64)
            check_attention(got, ref, dtype)
        else:   # the oracle's cache only needs the appended rows
            for i in range(len(seqs)):
                kc[:, :, i * host_cap + o_lens[i]] = nk_h[:, i]
                vc[:, :, i * host_cap + o_lens[i]] = nv_h[:, i]
            o_lens += 1
    torch.cuda.synchronize()
    ro.check_status()
    assert np.array_equal(ro.cache.lens.cpu().numpy(), budget_np + steps)
    final = SampledSeqs(ro.cache, seqs, host_cap)
    for i in range(len(seqs)):
        sl = slice(i * host_cap, i * host_cap + int(o_lens[i]))
        assert np.array_equal(final.k[:, :, sl], kc[:, :, sl]) and np.array_equal(final.v[:, :, sl], vc[:, :, sl])


def test_config1_tiny_fp32_every_step_every_sequence():
    run_round_and_decode(1, check_steps=list(range(64)), seqs=(0, 1, 2, 3))


def run_round_and_decode_every_sequence(cfg_id, check_steps):
    """Configs with one shared eviction list at full size, EVERY sequence: kept sets, orders and log-probs for all
    lists as above; then, one layer at a time streamed through host memory, the oracle takes the layer as it was
    generated (the per-plane seeds give the same bytes again), evicts with its own kept lists, appends the new rows of
    every decode step and recomputes attention for all sequences at ``check_steps``; at the end the whole layer
    (compacted rows and appended rows, every live row of every sequence) must equal the device's bit for bit.
    Nothing the oracle reads comes from the CUDA path: only seeded inputs and its own results."""
    b = ngc()
    from paper_2604_18002_b200.rollout import NgcRollout
    cfg = synth.CONFIGS[cfg_id]
    assert cfg["lists"] == 0
    L, Hq, Hkv, d, B, steps = cfg["L"], cfg["Hq"], cfg["Hkv"], cfg["d"], cfg["B"], cfg["steps"]
    dtype, dev = torch.bfloat16, "cuda"
    if isinstance(cfg["T"], tuple):
        lens = synth.ragged_lens(B, cfg["T"][0], cfg["T"][1], cfg["len_seed"])
    else:
        lens = torch.full((B,), cfg["T"], dtype=torch.int32)
    budget = torch.ceil(lens.double() / 3).to(torch.int32) if cfg["budget"] == "third" else \
        torch.full((B,), cfg["budget"], dtype=torch.int32)
    cap = torch.maximum(lens.long(), budget.long() + steps)
    n_max, k_max = int(lens.max()), int(budget.max())
    gen = dict(L=L, B=B, Hq=Hq, Hkv=Hkv, d=d, dtype=dtype, lens=lens, capacity=cap, seed=cfg["data_seed"],
               outlier_channels=cfg["outliers"], device=dev)
    src = synth.make_cache(**gen)
    ro = NgcRollout(L, B, Hq, Hkv, d, dtype, capacity=cap, n_max=n_max, k_max=k_max, lists=0, device=dev,
                    with_score=False, kv=(src.k, src.v))
    ro.cache.lens.copy_(src.lens)
    so = src.seq_off.cpu().numpy()
    del src
    logits = synth.make_logits(B, 1, n_max, seed=cfg["data_seed"] + 7, std=cfg["logit_std"], device=dev)
    n_t, k_t = lens.to(dev), budget.to(dev)
    ro.eviction_round(n_t, None, k_t, cfg["noise_seed"], 0, logits=logits)
    torch.cuda.synchronize()
    ro.check_status()

    # ---- sample and log-prob: every list
    lg, lens_np, budget_np = logits.cpu().numpy(), lens.numpy(), budget.numpy()
    r_ko, r_ks, _, r_st = oracle.sample_evict(lg, lens_np, None, budget_np, k_max, seed=cfg["noise_seed"], rnd=0)
    assert not r_st.any()
    assert np.array_equal(ro.kept_order.cpu().numpy(), r_ko), "kept_order differs"
    assert np.array_equal(ro.kept_sorted.cpu().numpy(), r_ks), "kept_sorted differs"
    ref_scan, rc = oracle.evict_logprob_scan(lg, lens_np, None, budget_np, r_ko)
    assert rc == 0 and np.max(np.abs(ro.logp.cpu().numpy() - ref_scan)) <= 1e-3
    assert np.array_equal(ro.cache.lens.cpu().numpy(), budget_np)

    # ---- decode on the GPU: all steps, whole batch; keep what the oracle will need (seeded inputs) and the outputs
    check_steps = sorted(set(check_steps))
    nk_all = np.empty((steps, L, B, Hkv, d), np.uint16)
    nv_all = np.empty((steps, L, B, Hkv, d), np.uint16)
    q_chk, out_chk = {}, {}
    out = torch.empty((L, B, Hq, d), dtype=torch.float32, device=dev)
    for s in range(steps):
        q = synth.make_queries(L, B, Hq, d, dtype, seed=1000 + s, device=dev)
        nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=5000 + 2 * s, device=dev)
        ro.decode_step(q, out, nk, nv)
        nk_all[s], nv_all[s] = synth.to_numpy(nk), synth.to_numpy(nv)
        if s in check_steps:
            q_chk[s], out_chk[s] = synth.to_numpy(q), out.cpu().numpy().astype(np.float64)
    torch.cuda.synchronize()
    ro.check_status()
    final_lens = budget_np + steps
    assert np.array_equal(ro.cache.lens.cpu().numpy(), final_lens)
    live = np.zeros(int(so[-1]), bool)                       # rows that hold a live token at the end
    for bb in range(B):
        live[so[bb]:so[bb] + final_lens[bb]] = True

    # ---- the oracle, layer by layer
    worst = 0.0
    for l in range(L):
        pre = synth.make_cache(**gen, layers=[l])
        kc, vc, nl, rc = oracle.compact_kv(synth.to_numpy(pre.k), synth.to_numpy(pre.v), so, lens_np, r_ks, budget_np, 0)
        del pre
        assert rc == 0 and np.array_equal(nl, budget_np)
        o_lens = nl.copy()
        for s in range(steps):
            if s in check_steps:
                ref, rc = oracle.decode_attn(kc, vc, so, o_lens, q_chk[s][l:l + 1], nk_all[s, l:l + 1], nv_all[s, l:l + 1])
                assert rc == 0                                # appends the step's rows and advances o_lens
                err = max_rel_err_per_vector(out_chk[s][l], ref[0])
                worst = max(worst, err)
                assert err <= 2e-2, (l, s, err)
            else:
                rows = so[:-1] + o_lens
                kc[0][:, rows] = nk_all[s, l].transpose(1, 0, 2)
                vc[0][:, rows] = nv_all[s, l].transpose(1, 0, 2)
                o_lens += 1
        assert np.array_equal(o_lens, final_lens)
        kg, vg = synth.to_numpy(ro.cache.k[l]), synth.to_numpy(ro.cache.v[l])
        assert np.array_equal(kg[:, live], kc[0][:, live]), f"K rows of layer {l} differ"
        assert np.array_equal(vg[:, live], vc[0][:, live]), f"V rows of layer {l} differ"
    print(f"config {cfg_id}: {B} sequences x {L} layers, attention at steps {check_steps}: worst rel err {worst:.2e}")


def test_config2_gqa_b64_full_size():
    need_gpu_gb(12)
    run_round_and_decode_every_sequence(2, check_steps=[0, 128, 255])


def test_config3_ragged_b256_full_size():
    need_gpu_gb(90)
    run_round_and_decode_every_sequence(3, check_steps=[0, 64, 127])


def test_config4_per_head_b128_full_size():
    need_gpu_gb(80)
    run_round_and_decode(4, seqs=(5,), check_steps=[0, 63], literal_lists=4)


def test_config5_rollout_loop_and_logprob_recompute():
    """Grow-then-evict loop: 256 prompt tokens, a round every 512 generated tokens down to 256
    (peak 768 = delta/epsilon of the steady-state proposition), 16 rounds; then all rounds'
    log-probs recomputed in one call from the stored logits and kept orders."""
    need_gpu_gb(8)
    b = ngc()
    from paper_2604_18002_b200.rollout import NgcRollout
    cfg = synth.CONFIGS[5]
    L, Hq, Hkv, d, B = cfg["L"], cfg["Hq"], cfg["Hkv"], cfg["d"], cfg["B"]
    prompt, cadence, K, rounds = cfg["T"], cfg["cadence"], cfg["budget"], cfg["steps"] // cfg["cadence"]
    peak = prompt + cadence
    dtype, dev, lists = torch.bfloat16, "cuda", cfg["lists"]
    src = synth.make_cache(L, B, Hq, Hkv, d, dtype, [prompt] * B, capacity=peak, seed=3, device=dev)
    ro = NgcRollout(L, B, Hq, Hkv, d, dtype, capacity=peak, n_max=peak, k_max=K, lists=lists, device=dev, with_score=False,
                    kv=(src.k, src.v))
    G = ro.G
    ro.cache.lens.copy_(src.lens)
    del src
    seqs = [0, 41]
    mirror = SampledSeqs(ro.cache, seqs, peak)
    kc, vc = mirror.k, mirror.v
    o_lens = np.full(len(seqs), prompt, np.int32)
    all_logits = torch.empty((rounds, B, G, peak), dtype=torch.float32, device=dev)
    all_ko = torch.empty((rounds, B, G, K), dtype=torch.int32, device=dev)
    all_lp = torch.empty((rounds, B, G), dtype=torch.float64, device=dev)
    n_t = torch.full((B,), peak, dtype=torch.int32, device=dev)
    k_t = torch.full((B,), K, dtype=torch.int32, device=dev)
    out = torch.empty((L, B, Hq, d), dtype=torch.float32, device=dev)
    check_in_round = {0: [0, 511], 7: [100], 15: [511]}
    step = 0
    for r in range(rounds):
        for s in range(cadence):
            q = synth.make_queries(L, B, Hq, d, dtype, seed=20000 + step, device=dev)
            nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=40000 + 2 * step, device=dev)
            ro.decode_step(q, out, nk, nv)
            nk_h, nv_h = synth.to_numpy(nk[:, seqs]), synth.to_numpy(nv[:, seqs])
            if s in check_in_round.get(r, []):
                ref, rc = oracle.decode_attn(kc, vc, mirror.so, o_lens, synth.to_numpy(q[:, seqs]), nk_h, nv_h)
                assert rc == 0
                check_attention(out[:, seqs].cpu().numpy().astype(np.float64), ref, dtype)
            else:
                for i in range(len(seqs)):
                    kc[:, :, i * peak + o_lens[i]] = nk_h[:, i]
                    vc[:, :, i * peak + o_lens[i]] = nv_h[:, i]
                o_lens += 1
            step += 1
        # cache is at its peak (the steady state delta/epsilon = 512 / (2/3) = 768): evict down to K
        assert int(ro.cache.lens.max()) == peak and int(ro.cache.lens.min()) == peak
        all_logits[r] = synth.make_logits(B, G, peak, seed=60000 + r, device=dev)
        ro.eviction_round(n_t, None, k_t, cfg["noise_seed"], r, logits=all_logits[r])
        all_ko[r] = ro.kept_order
        all_lp[r] = ro.logp[0]
        lg = all_logits[r, seqs].cpu().numpy()
        r_ko, r_ks, _, st = oracle.sample_evict(lg[:1], [peak], None, [K], K, seed=cfg["noise_seed"], rnd=r, list_base=seqs[0] * G)
        r_ko2, r_ks2, _, _ = oracle.sample_evict(lg[1:], [peak], None, [K], K, seed=cfg["noise_seed"], rnd=r, list_base=seqs[1] * G)
        r_ks = np.concatenate([r_ks, r_ks2])
        assert np.array_equal(ro.kept_order[seqs].cpu().numpy(), np.concatenate([r_ko, r_ko2]))
        kc, vc, nl, rc = oracle.compact_kv(kc, vc, mirror.so, o_lens, r_ks, [K, K], lists)
        assert rc == 0
        o_lens = nl.copy()
    torch.cuda.synchronize()
    ro.check_status()
    assert np.array_equal(ro.cache.lens.cpu().numpy(), np.full(B, K, np.int32))
    final = SampledSeqs(ro.cache, seqs, peak)
    for i in range(len(seqs)):
        sl = slice(i * peak, i * peak + K)
        assert np.array_equal(final.k[:, :, sl], kc[:, :, sl]) and np.array_equal(final.v[:, :, sl], vc[:, :, sl])
    # ---- policy-gradient recompute: every round's log-prob in one call
    lp2 = torch.empty((rounds, B, G), dtype=torch.float64, device=dev)
    st = b.new_status()
    n_all = torch.full((rounds, B), peak, dtype=torch.int32, device=dev)
    k_all = torch.full((rounds, B), K, dtype=torch.int32, device=dev)
    b.ngc_evict_logprob(all_logits, n_all, None, k_all, all_ko, lp2, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert torch.equal(lp2, all_lp)                       # same kernel, same inputs: identical bits
    lg = all_logits.cpu().numpy()
    ko = all_ko.cpu().numpy()
    n_np, k_np = np.full((rounds, B), peak, np.int32), np.full((rounds, B), K, np.int32)
    ref, rc = oracle.evict_logprob_scan(lg, n_np, None, k_np, ko)
    assert rc == 0 and np.max(np.abs(lp2.cpu().numpy() - ref)) <= 1e-3
    # Eq. (1) literally on a spread of (round, sequence) pairs, all their layers' lists
    for r, bb in [(0, 0), (5, 17), (15, 63)]:
        lit, rc = oracle.evict_logprob(lg[r, bb:bb + 1], [peak], None, [K], ko[r, bb:bb + 1])
        assert rc == 0 and np.max(np.abs(lp2[r, bb].cpu().numpy() - lit[0, 0])) <= 1e-3


def test_config6_paper_setting_block_eviction_scored_from_k():
    """The paper's own eviction setting at full size (Section 5.1: units of 32 tokens, 5 recent queries,
    a round every 256 tokens keeping half, one list per layer): 512 rollouts, 4 rounds.  Every round's
    scores are checked on sampled sequences (2e-2 of the largest score), the draw for EVERY list
    bit-exact from the scores the GPU produced, Eq. (1) literally for every list, the compacted rows
    of the sampled sequences bit-exact, attention at a few steps."""
    need_gpu_gb(12)
    b = ngc()
    from paper_2604_18002_b200.rollout import NgcRollout
    cfg = synth.CONFIGS[6]
    L, Hq, Hkv, d, B = cfg["L"], cfg["Hq"], cfg["Hkv"], cfg["d"], cfg["B"]
    prompt, cadence, K, block = cfg["T"], cfg["cadence"], cfg["budget"], cfg["block"]
    rounds = cfg["steps"] // cadence
    peak = prompt + cadence
    N = peak // block
    dtype, dev, lists, w = torch.bfloat16, "cuda", cfg["lists"], 5
    src = synth.make_cache(L, B, Hq, Hkv, d, dtype, [prompt] * B, capacity=peak, seed=4, device=dev)
    ro = NgcRollout(L, B, Hq, Hkv, d, dtype, capacity=peak, n_max=N, k_max=K, lists=lists, block=block, w=w, device=dev,
                    kv=(src.k, src.v))
    G = ro.G
    ro.cache.lens.copy_(src.lens)
    del src
    seqs = [0, 300]
    mirror = SampledSeqs(ro.cache, seqs, peak)
    kc, vc = mirror.k, mirror.v
    o_lens = np.full(len(seqs), prompt, np.int32)
    n_np, k_np = np.full(B, N, np.int32), np.full(B, K, np.int32)
    n_t, k_t = torch.as_tensor(n_np).to(dev), torch.as_tensor(k_np).to(dev)
    out = torch.empty((L, B, Hq, d), dtype=torch.float32, device=dev)
    check_in_round = {0: [0, 255], 2: [77], 3: [255]}
    step = 0
    for r in range(rounds):
        for s in range(cadence):
            q = synth.make_queries(L, B, Hq, d, dtype, seed=20000 + step, device=dev)
            nk, nv = synth.make_new_kv(L, B, Hkv, d, dtype, seed=40000 + 2 * step, device=dev)
            ro.decode_step(q, out, nk, nv)
            nk_h, nv_h = synth.to_numpy(nk[:, seqs]), synth.to_numpy(nv[:, seqs])
            if s in check_in_round.get(r, []):
                ref, rc = oracle.decode_attn(kc, vc, mirror.so, o_lens, synth.to_numpy(q[:, seqs]), nk_h, nv_h)
                assert rc == 0
                check_attention(out[:, seqs].cpu().numpy().astype(np.float64), ref, dtype)
            else:
                for i in range(len(seqs)):
                    kc[:, :, i * peak + o_lens[i]] = nk_h[:, i]
                    vc[:, :, i * peak + o_lens[i]] = nv_h[:, i]
                o_lens += 1
            step += 1
        assert int(ro.cache.lens.max()) == peak and int(ro.cache.lens.min()) == peak
        qr = synth.normal((L, B, Hq, w, d), 70000 + r, dtype, device=dev)
        ro.eviction_round(n_t, None, k_t, cfg["noise_seed"], r, q_recent=qr)          # draws from the scores
        torch.cuda.synchronize()
        ro.check_status()
        lg = ro.logits.cpu().numpy()
        # scores of the sampled sequences
        ref_s = oracle.score_evict(kc, mirror.so, o_lens, synth.to_numpy(qr[:, seqs]), block, lists, n_max=N)
        for i, bb in enumerate(seqs):
            for g in range(G):
                assert np.max(np.abs(lg[bb, g] - ref_s[i, g])) <= 2e-2 * ref_s[i, g].max()
            assert abs(lg[bb].sum() * block - G) <= 1e-2                                # each layer's psi sums to one
        # the draw, every list, from the very logits the GPU wrote
        r_ko, r_ks, _, st = oracle.sample_evict(lg, n_np, None, k_np, K, seed=cfg["noise_seed"], rnd=r)
        assert not st.any()
        assert np.array_equal(ro.kept_order.cpu().numpy(), r_ko) and np.array_equal(ro.kept_sorted.cpu().numpy(), r_ks)
        lit, rc = oracle.evict_logprob(lg, n_np, None, k_np, r_ko)
        assert rc == 0 and np.max(np.abs(ro.logp.cpu().numpy() - lit)) <= 1e-3
        sel = np.array(seqs)
        kc, vc, nl, rc = oracle.compact_kv(kc, vc, mirror.so, o_lens, r_ks[sel], k_np[sel], lists, block)
        assert rc == 0 and np.all(nl == K * block)
        o_lens = nl.copy()
        after = SampledSeqs(ro.cache, seqs, peak)
        for i in range(len(seqs)):
            sl = slice(i * peak, i * peak + K * block)
            assert np.array_equal(after.k[:, :, sl], kc[:, :, sl]) and np.array_equal(after.v[:, :, sl], vc[:, :, sl])
    assert np.array_equal(ro.cache.lens.cpu().numpy(), np.full(B, K * block, np.int32))     # steady state: delta / epsilon / 2


def test_score_backward_config2_shape_sampled_sequences():
    """Gradient of the scores at the benchmark's cache shape (B = 64, T = 4096, 12/2 heads, shared list; 4 of the 28
    layers to keep the oracle to seconds): two sampled sequences against the oracle, 2e-2 of the largest entry."""
    need_gpu_gb(6)
    b = ngc()
    cfg = synth.CONFIGS[2]
    L, Hq, Hkv, d, B, T, w = 4, cfg["Hq"], cfg["Hkv"], cfg["d"], cfg["B"], cfg["T"], 5
    dev, dtype = "cuda", torch.bfloat16
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, [T] * B, capacity=T, seed=8, outlier_channels=4, device=dev)
    dc = b.NgcCache(c.k, c.v, c.seq_off, c.lens, Hq, T)
    qr = synth.normal((L, B, Hq, w, d), 9, dtype, device=dev)
    up = synth.make_logits(B, 1, T, seed=10, device=dev)
    gq = torch.empty(qr.shape, dtype=torch.float32, device=dev)
    gk = torch.zeros_like(c.k)
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_SCORE_BACKWARD, dc))
    st = b.new_status()
    b.ngc_score_evict_backward(dc, qr, 1, b.LISTS_SHARED, up, gq, gk, ws=ws, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    for bb in (0, 63):
        k1 = synth.to_numpy(c.k[:, :, bb * T:(bb + 1) * T])
        ref_q, ref_k = oracle.score_evict_grad(k1, np.array([0, T], np.int64), np.array([T], np.int32), synth.to_numpy(qr[:, bb:bb + 1]), 1, 0,
                                               up[bb:bb + 1].cpu().numpy().astype(np.float64))
        got_q = gq[:, bb:bb + 1].cpu().numpy().astype(np.float64)
        got_k = synth.as_f64(synth.to_numpy(gk[:, :, bb * T:(bb + 1) * T]))
        assert np.max(np.abs(got_q - ref_q)) <= 2e-2 * np.abs(ref_q).max() + 1e-6
        assert np.max(np.abs(got_k - ref_k)) <= 2e-2 * np.abs(ref_k).max() + 1e-6


def test_replay_attn_rollout_loop_history_sampled_sequence():
    """Replay attention over the rollout-loop history (T = 8448, 16 rounds, 768 -> 256 per round, per-layer lists),
    one layer, B = 8: sequence 5 against the dense-mask oracle at all of its 8448 positions."""
    need_gpu_gb(4)
    b = ngc()
    from oracle import replay
    cfg = synth.CONFIGS[5]
    L, Hq, Hkv, d, B = 1, cfg["Hq"], cfg["Hkv"], cfg["d"], 8
    K, delta, prompt = cfg["budget"], cfg["cadence"], cfg["T"]
    R, alive = cfg["steps"] // delta, prompt + delta
    T = prompt + R * delta
    dev, dtype = "cuda", torch.bfloat16
    rng = np.random.default_rng(4)
    ks = np.sort(np.argsort(rng.random((R, B, L, alive)), -1)[..., :K], -1).astype(np.int32)
    budget = np.full((R, B), K, np.int32)
    alive_before = np.full((R, B), alive, np.int32)
    total_before = (alive + delta * np.arange(R))[:, None].repeat(B, 1).astype(np.int32)
    t = lambda a: torch.as_tensor(a).to(dev)
    pos = torch.empty((R, B, L, K), dtype=torch.int32, device=dev)
    cnt = torch.empty((R, B, L), dtype=torch.int32, device=dev)
    st = b.new_status()
    b.ngc_replay_visibility(t(ks), t(budget), t(alive_before), t(total_before), 1, alive, pos, cnt, status=st)
    c = synth.make_cache(L, B, Hq, Hkv, d, dtype, [T] * B, capacity=T, seed=6, device=dev)
    dc = b.NgcCache(c.k, c.v, c.seq_off, c.lens, Hq, T)
    q = synth.normal((L, B, Hq, T, d), 7, dtype, device=dev)
    out = torch.empty((L, B, Hq, T, d), dtype=torch.float32, device=dev)
    b.ngc_replay_attn(dc, q, out, pos, cnt, t(total_before), lists=b.LISTS_PER_LAYER, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    bb = 5
    ref_pos, ref_cnt, rc = replay.alive_positions(ks[:, bb:bb + 1], budget[:, bb:bb + 1], alive_before[:, bb:bb + 1], total_before[:, bb:bb + 1])
    assert rc == 0 and np.array_equal(pos[:, bb:bb + 1].cpu().numpy(), ref_pos)
    M = replay.dense_mask(T, [int(x) for x in total_before[:, bb]], [ref_pos[r, 0, 0, : ref_cnt[r, 0, 0]] for r in range(R)])
    ref = replay.replay_attention(synth.as_f64(synth.to_numpy(q[0, bb])), synth.as_f64(synth.to_numpy(c.k[0, :, bb * T:(bb + 1) * T])),
                                  synth.as_f64(synth.to_numpy(c.v[0, :, bb * T:(bb + 1) * T])), M[None])
    assert max_rel_err_per_vector(out[0, bb].cpu().numpy().astype(np.float64), ref) <= 2e-2
