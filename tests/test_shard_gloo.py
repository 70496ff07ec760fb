"""The N>1 path on CPU: two gloo ranks shard the sequences, run the eviction path (the oracle stands in for the
device here) on their shard only, and the gathered result equals the single-process run; the throughput
reduction takes the sum of units and the max of times."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_16187_b200 import shard
from paper_2412_16187_b200 import workloads as wl


def test_shard_range_is_a_partition():
    for n, world in [(64, 8), (5, 2), (3, 4), (16, 1), (7, 3)]:
        got = [shard.shard_range(n, r, world) for r in range(world)]
        assert got[0][0] == 0 and got[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(got, got[1:]))
        sizes = [hi - lo for lo, hi in got]
        assert max(sizes) - min(sizes) <= 1


def _run_shard(w, lo, hi):
    import oracle

    n = hi - lo
    Nmax = w.max_prompt_len
    W = wl.gen_W(w)
    K, Q, V = (wl.gen_tokens(w, x, lo, n, 0, Nmax) for x in "kqv")
    oc = oracle.OracleCache(n, w.n_kv_heads, w.group_size, w.head_dim, w.hash_bits, w.max_budget, w.budgets()[lo:hi],
                            w.dtype)
    oc.prefill(W, Q, K, V, w.prompt_lens()[lo:hi])
    return oc.pos.copy(), oc.codes.copy()


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.CONFIGS["throughput_batch"].scaled(batch=5, budget_lo=24, budget_hi=80, decode_steps=0)
    lo, hi = shard.shard_range(w.n_seq, rank, world)
    pos, codes = _run_shard(w, lo, hi)
    gathered = [None] * world
    dist.all_gather_object(gathered, (lo, hi, pos, codes))
    units, secs, rate = shard.job_throughput(float((hi - lo) * w.n_kv_heads), 1.0 + rank)  # rank 1 is "slower"
    if rank == 0:
        full_pos, full_codes = _run_shard(w, 0, w.n_seq)
        ok = all(np.array_equal(full_pos[a:b], p) and np.array_equal(full_codes[a:b], c) for a, b, p, c in gathered)
        out.put((ok, units, secs, rate, w.n_units))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_without_exchanging_data():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ok, units, secs, rate, n_units = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok
    assert units == n_units and secs == 2.0 and rate == n_units / 2.0
