"""Multi-rank path on CPU (gloo, world size 2): batch sharding needs no data-path
collective, and a sharded batch draws the keep sets of the unsharded batch
because Philox list indices are global.  The ranks run the CPU oracle here; on
GPUs the same host logic drives the CUDA library (bench.py --gpus N)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_18002_b200 import synth
from paper_2604_18002_b200.sharding import list_base, shard_batch


def test_shard_batch_balances_and_covers():
    lens = synth.ragged_lens(256, 1024, 8192, 2).tolist()
    for world in (1, 2, 3, 8):
        rs = shard_batch(lens, world)
        assert rs[0][0] == 0 and rs[-1][1] == 256 and all(a[1] == b[0] for a, b in zip(rs, rs[1:]))
        sums = [sum(lens[a:b]) for a, b in rs]
        assert all(b > a for a, b in rs)
        assert max(sums) <= 1.05 * sum(lens) / world + max(lens)
    assert shard_batch([5, 5], 4) == [(0, 1), (1, 2), (2, 2), (2, 2)]
    assert shard_batch([], 2) == [(0, 0), (0, 0)]
    with pytest.raises(ValueError):
        shard_batch([1], 0)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, G, n_max = 12, 3, 200
        lens = synth.ragged_lens(B, 50, 200, 2).numpy()
        budget = (lens // 2).astype(np.int32)
        logits = synth.make_logits(B, G, n_max, seed=4).numpy()
        a, b = shard_batch(lens.tolist(), world)[rank]
        ko, ks, _, st = oracle.sample_evict(logits[a:b], lens[a:b], None, budget[a:b], 100, seed=9, rnd=3,
                                            list_base=list_base((a, b), G))
        assert not st.any()
        lp, _ = oracle.evict_logprob(logits[a:b], lens[a:b], None, budget[a:b], ko)
        # bench.py's only communication: a barrier and the max over ranks of the timed region
        dist.barrier()
        t = torch.tensor([float(rank + 1)], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == world
        gathered = [None] * world
        dist.all_gather_object(gathered, (a, b, ko, ks, lp))
        if rank == 0:
            full_ko, full_ks, _, _ = oracle.sample_evict(logits, lens, None, budget, 100, seed=9, rnd=3)
            full_lp, _ = oracle.evict_logprob(logits, lens, None, budget, full_ko)
            cover = 0
            for (ga, gb, gko, gks, glp) in gathered:
                assert np.array_equal(gko, full_ko[ga:gb]) and np.array_equal(gks, full_ks[ga:gb])
                assert np.array_equal(glp[0], full_lp[0, ga:gb])
                cover += gb - ga
            assert cover == B
            q.put("ok")
    finally:
        dist.destroy_process_group()


def test_sharded_equals_unsharded_world2_gloo():
    import oracle
    oracle.build()          # compile once in the parent, not concurrently in the children
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert q.get(timeout=5) == "ok"
