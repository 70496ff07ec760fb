#!/usr/bin/env python
"""Benchmark of the HashEvict eviction hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One bench step = one pass of the whole hot path over one batch of synthetic input: for every layer replica,
he_prefill_compress of the prompt batch, then T decode steps, each of which calls he_decode_step once per layer
replica (layer by layer, as a model would). The decode calls of a step are captured once into a CUDA graph (the
library neither allocates nor synchronises) and replayed, so the timing is the GPU's, not the Python loop's.

Printed: ONE JSON line. `value` is decode evictions/s (unit-steps per second over all GPUs, inputs resident in
HBM); prefill keys/s, the roofline fractions, the end-to-end number through the host-buffer entry points and the
CPU oracle's speed on a bounded sample are further keys of the same line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2412_16187_b200 import workloads as wl  # noqa: E402

METRIC = "decode evictions/s (seq x KV-head steps)"
UNIT = "evictions/s"
DEFAULT_REPLICAS = {"throughput_batch": 16, "long_prefill": 8, "llama3_8b_gqa": 64, "llama2_7b_layer": 128, "tiny": 4}
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------------- bytes

def decode_bytes_per_call(w, budgets, write_scores=True):
    """Algorithmic bytes one he_decode_step call must move (all units evicting): new q/k/v rows in, codes in,
    scores out, the victim slot's K/V/code/pos out, victim index out, W once."""
    d, e, G, b = w.head_dim, w.elem_bytes, w.group_size, w.hash_bits
    per_unit_fixed = (G + 2) * d * e + 2 * d * e + b / 8 + 8
    per_slot = b / 8 + (4 if write_scores else 0)
    slots = float(np.sum(budgets.astype(np.int64))) * w.n_kv_heads
    return w.n_units * per_unit_fixed + slots * per_slot + d * b * 4


def prefill_bytes_per_call(w, budgets, plens):
    """Algorithmic bytes of one he_prefill_compress call: K hashed once, Q rows of evicting tokens hashed once,
    surviving K/V read and written once, code/pos/score tables written."""
    d, e, G, b, H = w.head_dim, w.elem_bytes, w.group_size, w.hash_bits, w.n_kv_heads
    N = plens.astype(np.int64)
    C = np.minimum(budgets.astype(np.int64), N)
    per_seq = N * d * e + (N - C) * G * d * e + 2 * C * d * e + 2 * C * d * e + C * (b / 8 + 8)
    return float(per_seq.sum()) * H


NOMINAL_HBM_GBS = 8000.0  # the vendor's figure, for context beside the measured copy bandwidth
RESOLVER_CYCLES_PER_STEP = 144.0  # one warp walking Algorithm 1's evicting steps in order (measured in isolation)


def profiled_traffic(kernel, workload):
    """DRAM bytes per launch of `kernel` from the committed ncu summary profiles/<kernel>_<workload>.md (its line
    'dram bytes per launch: N'), or None when there is no such summary."""
    import re

    path = os.path.join(ROOT, "profiles", f"{kernel}_{workload}.md")
    if not os.path.exists(path):
        return None, None
    m = re.search(r"dram bytes per launch[^0-9]*([0-9][0-9_,]*)", open(path).read())
    return (int(m.group(1).replace(",", "").replace("_", "")) if m else None), os.path.relpath(path, ROOT)


def replay_bounds(w, budgets, plens, sms, sm_mhz):
    """What bounds Section 3's sequential prompt replay in this design: every evicting step of a unit passes through
    one resolver warp (a dependent chain of RESOLVER_CYCLES_PER_STEP cycles), one unit per SM at a time."""
    N = plens.astype(np.int64)
    C = np.minimum(budgets.astype(np.int64), N)
    steps = float((N - C).sum()) * w.n_kv_heads  # evicting steps of one call, all units
    clock = (sm_mhz or 1965.0) * 1e6
    return steps, sms * clock / RESOLVER_CYCLES_PER_STEP  # steps per call, steps per second at the chain's pace


# ------------------------------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        fd, self.path = tempfile.mkstemp(suffix=".csv")
        os.close(fd)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r.split(", ") for r in open(self.path).read().strip().splitlines() if r.count(",") >= 6]
        os.unlink(self.path)
        if not rows:
            return out
        sm = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].strip() == "Active" for r in rows)]
        out.update(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=float(rows[0][1]), reasons=reasons,
                   samples=len(rows), power_w_max=max(float(r[2]) for r in rows))
        return out


# ------------------------------------------------------------------------------------------------- oracle legs

def oracle_sample(w, seqs, decode_steps, threads):
    """Times the CPU oracle, as it stands, on the first `seqs` sequences: prefill then `decode_steps` steps."""
    import oracle

    seqs = min(seqs, w.n_seq)
    budgets, plens = w.budgets()[:seqs], w.prompt_lens()[:seqs]
    Nmax = int(plens.max())
    W = wl.gen_W(w)
    K = np.zeros((seqs, w.n_kv_heads, Nmax, w.head_dim), dtype=wl.np_dtype(w))
    V = np.zeros_like(K)
    Q = np.zeros((seqs, w.n_kv_heads * w.group_size, Nmax, w.head_dim), dtype=wl.np_dtype(w))
    for s in range(seqs):
        n = int(plens[s])
        K[s, :, :n] = wl.gen_tokens(w, "k", s, 1, 0, n)[0]
        V[s, :, :n] = wl.gen_tokens(w, "v", s, 1, 0, n)[0]
        Q[s, :, :n] = wl.gen_tokens(w, "q", s, 1, 0, n)[0]
    cmax = (int(budgets.max()) + 3) // 4 * 4
    oc = oracle.OracleCache(seqs, w.n_kv_heads, w.group_size, w.head_dim, w.hash_bits, cmax, budgets, w.dtype,
                            n_sink=w.n_sink, n_recent=w.n_recent, threads=threads)
    t0 = time.perf_counter()
    oc.prefill(W, Q, K, V, plens)
    t_prefill = time.perf_counter() - t0
    dq = wl.gen_decode_inputs(w, "q", 0, decode_steps)[:, :seqs]
    dk = wl.gen_decode_inputs(w, "k", 0, decode_steps)[:, :seqs]
    dv = wl.gen_decode_inputs(w, "v", 0, decode_steps)[:, :seqs]
    t0 = time.perf_counter()
    for i in range(decode_steps):
        oc.step(W, np.ascontiguousarray(dq[i]), np.ascontiguousarray(dk[i]), np.ascontiguousarray(dv[i]))
    t_decode = time.perf_counter() - t0
    units = seqs * w.n_kv_heads
    return {
        "evictions_per_s": units * decode_steps / t_decode,
        "prefill_keys_per_s": float(plens.sum()) * w.n_kv_heads / t_prefill,
        "t_prefill_s": t_prefill, "t_decode_s": t_decode,
        "sample": f"first {seqs} of {w.n_seq} sequences ({units} units): full prefill, then {decode_steps} decode steps",
    }


def run_reference(args, w):
    """--impl reference: the oracle timed on the host cores, same metric and config."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = len(os.sched_getaffinity(0))
    seqs, dsteps = args.ref_seqs, args.ref_decode_steps
    vals, pf = [], []
    for i in range(args.warmup + args.steps):
        r = oracle_sample(w, seqs, dsteps, threads)
        if i >= args.warmup:
            vals.append(r["evictions_per_s"])
            pf.append(r["prefill_keys_per_s"])
    v = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * (r["t_prefill_s"] + r["t_decode_s"]), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": config_dict(w, args.replicas),
        "prefill_keys_per_s": statistics.mean(pf),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": r["sample"]},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


PACKED_CODES = False  # set from --packed-codes


def config_dict(w, replicas):
    return {
        "workload": w.name, "batch": w.batch, "layers_folded": w.layers, "n_kv_heads": w.n_kv_heads,
        "group_size": w.group_size, "head_dim": w.head_dim, "hash_bits": w.hash_bits, "kv_dtype": w.dtype,
        "budget": "ragged U[%d,%d]" % (w.budget_lo, w.budget_hi) if w.ragged else w.budget,
        "prompt_len": "%d x budget" % w.prompt_factor if w.ragged else w.prompt_len,
        "decode_steps": w.decode_steps, "layer_replicas": replicas, "n_sink": w.n_sink, "n_recent": w.n_recent,
        "write_scores": True, "packed_codes": bool(PACKED_CODES),
        "l2": "inputs larger than L2: every decode call streams a different layer replica's tables "
              "(replicas x per-call bytes > 126 MB); prefill reads GBs of prompt",
    }


# ------------------------------------------------------------------------------------------------- ours

def run_ours(args, w):
    import torch
    import torch.distributed as dist

    from paper_2412_16187_b200 import HashEvictCache, decode_staging_bytes

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    # weak scaling: every rank runs the same shapes on its own seeded shard (independent sequences, no collective)
    w = w.scaled(seed=w.seed + 1000 * rank)
    R, T = args.replicas, w.decode_steps
    B, H, G, d = w.n_seq, w.n_kv_heads, w.group_size, w.head_dim
    budgets, plens = w.budgets(), w.prompt_lens()
    Nmax = w.max_prompt_len
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32

    def up(a):
        t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda(non_blocking=False)
        return t.view(torch.bfloat16) if a.dtype == np.uint16 else t

    # ---- inputs: generated on the host (seeded), uploaded once; the timed region starts with them in HBM
    t_gen = time.perf_counter()
    dK = torch.zeros((B, H, Nmax, d), dtype=tdt, device="cuda")
    dV = torch.zeros_like(dK)
    dQ = torch.zeros((B, H * G, Nmax, d), dtype=tdt, device="cuda")
    for s in range(B):
        n = int(plens[s])
        dK[s, :, :n] = up(wl.gen_tokens(w, "k", s, 1, 0, n)[0])
        dV[s, :, :n] = up(wl.gen_tokens(w, "v", s, 1, 0, n)[0])
        dQ[s, :, :n] = up(wl.gen_tokens(w, "q", s, 1, 0, n)[0])
    gq, gk, gv = (up(wl.gen_decode_inputs(w, x, 0, T)) for x in "qkv")
    dplen = torch.from_numpy(plens).cuda()
    caches = [HashEvictCache(B, H, G, d, w.hash_bits, budgets, torch.from_numpy(wl.gen_W(w, layer=r)), dtype=tdt,
                             n_sink=w.n_sink, n_recent=w.n_recent, write_scores=True, packed_codes=args.packed_codes,
                             early_inputs=not args.no_early_inputs)
              for r in range(R)]
    ws = caches[0].workspace(Nmax)
    victims = torch.empty((R, B, H), dtype=torch.int32, device="cuda")
    t_gen = time.perf_counter() - t_gen

    stream = torch.cuda.Stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def prefill_all():
        for c in caches:
            c.prefill_compress(dQ, dK, dV, dplen, Nmax, workspace=ws, stream=stream)

    def decode_all():
        for i in range(T):
            for r, c in enumerate(caches):
                c.decode_step(gq[i], gk[i], gv[i], victim_out=victims[r], stream=stream)

    # capture the T x R decode calls once; the library neither allocates nor synchronises, so it is capturable
    graph = None
    with torch.cuda.stream(stream):
        prefill_all()
        stream.synchronize()
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                decode_all()

    def one_step():
        e0, e1, e2 = ev(), ev(), ev()
        with torch.cuda.stream(stream):
            e0.record(stream)
            prefill_all()
            e1.record(stream)
            if graph is not None:
                graph.replay()
            else:
                decode_all()
            e2.record(stream)
        return e0, e1, e2

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t_wall = time.perf_counter()
    evs = [one_step() for _ in range(args.steps)]
    barrier()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop() if rank == 0 else None
    t_prefill = sum(e0.elapsed_time(e1) for e0, e1, _ in evs) * 1e-3
    t_decode = sum(e1.elapsed_time(e2) for _, e1, e2 in evs) * 1e-3
    from paper_2412_16187_b200 import shard

    K = args.steps
    units = w.n_units
    decode_calls = T * R * K
    # whole job = units of all ranks / max over ranks of the device time (no data-path collective: units are independent)
    evictions, t_decode, value = shard.job_throughput(float(units * T * R * K), t_decode, device="cuda")
    keys, t_prefill, prefill_rate = shard.job_throughput(float(plens.sum()) * H * R * K, t_prefill, device="cuda")
    t_total = t_prefill + t_decode
    peak, peak_src = measured_peak()
    dec_bytes = decode_bytes_per_call(w, budgets)
    pre_bytes = prefill_bytes_per_call(w, budgets, plens)
    dec_gbs = dec_bytes * decode_calls / t_decode / 1e9
    pre_gbs = pre_bytes * R * K / t_prefill / 1e9

    early = not args.no_early_inputs
    decode_kernel = "decode_step_sm_kernel" if (early and units <= 4 * 148 and not args.packed_codes and d % 32 == 0) else "decode_step_kernel"
    traffic, traffic_src = profiled_traffic(decode_kernel, w.name)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
        "ms_per_step": 1e3 * t_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u32", "data": "synthetic", "config": config_dict(w, R),
        "decode_us_per_call": 1e6 * t_decode / decode_calls,
        "decode_launch_mode": "cuda graph of he_decode_step calls" if graph is not None else "plain stream launches",
        "decode_inputs": "HE_FLAG_EARLY_INPUTS: q, k, v of all steps are staged in HBM before the graph is launched, so each call "
                         "may hash its rows under the previous call's scan" if early else "default order (rows read after the previous kernel ended)",
        "prefill_keys_per_s": prefill_rate, "prefill_ms_per_call": 1e3 * t_prefill / (R * K),
        "roofline": {"kernel": decode_kernel, "bound": "hbm", "achieved": dec_gbs, "peak": peak, "unit": "GB/s",
                     "frac": dec_gbs / peak, "peak_source": peak_src, "frac_of_nominal_8TBs": dec_gbs / NOMINAL_HBM_GBS,
                     "traffic": traffic, "traffic_source": traffic_src,
                     "algorithmic_bytes_per_launch": dec_bytes},
        "roofline_prefill": {"call": "he_prefill_compress (hash K, hash Q, replay, gather)", "bound": "hbm",
                             "achieved": pre_gbs, "peak": peak, "unit": "GB/s", "frac": pre_gbs / peak,
                             "frac_of_nominal_8TBs": pre_gbs / NOMINAL_HBM_GBS,
                             "algorithmic_bytes_per_call": pre_bytes,
                             "note": "the HBM fraction of the whole call, as the metric asks; Section 3's replay phase is a "
                                     "sequential dependent chain per unit, its own bound is in prefill_phases.replay_bound"},
        "gpu_launches": K * R * (6 + T),  # per prefill: W image, hash K, hash Q, schedule, replay, gather; per decode call: 1
        "input_setup_s": t_gen,
    }

    from paper_2412_16187_b200 import prefill_phase_events

    sms = torch.cuda.get_device_properties(local).multi_processor_count
    sm_mhz = clocks.get("sm_mhz") if clocks else None

    def phase_split(cache_list, dQ_, dK_, dV_, dplen_, Nmax_, ws_, reps=1):
        """Milliseconds per call of the phases of he_prefill_compress, from events the library records around them
        (the same kernels as in the timed region, one event record between two phases)."""
        evs5 = [[ev() for _ in range(5)] for _ in range(len(cache_list) * reps)]
        with torch.cuda.stream(stream):
            k = 0
            for _ in range(reps):
                for c in cache_list:
                    prefill_phase_events(evs5[k])
                    c.prefill_compress(dQ_, dK_, dV_, dplen_, Nmax_, workspace=ws_, stream=stream)
                    k += 1
            prefill_phase_events(None)
        torch.cuda.synchronize()
        names = ("hash_k_ms", "hash_q_ms", "schedule_replay_ms", "gather_ms")
        out = {n: statistics.mean(e[i].elapsed_time(e[i + 1]) for e in evs5) for i, n in enumerate(names)}
        out["call_ms"] = statistics.mean(e[0].elapsed_time(e[4]) for e in evs5)
        return out

    def replay_bound_obj(wk, budgets_, plens_, replay_ms):
        steps, peak_steps = replay_bounds(wk, budgets_, plens_, sms, sm_mhz)
        ach = steps / (replay_ms * 1e-3)
        return {"bound": "latency: one resolver warp per SM walks a unit's evicting steps in order, a dependent chain of "
                         f"{RESOLVER_CYCLES_PER_STEP:.0f} cycles per step", "unit": "evicting steps/s", "achieved": ach,
                "peak": peak_steps, "frac": ach / peak_steps, "evicting_steps_per_call": steps,
                "hbm_floor_ms_of_the_whole_call": None}

    if rank == 0 and not args.skip_phases:
        ph = phase_split(caches, dQ, dK, dV, dplen, Nmax, ws)
        ph["replay_bound"] = replay_bound_obj(w, budgets, plens, ph["schedule_replay_ms"])
        ph["replay_bound"]["hbm_floor_ms_of_the_whole_call"] = pre_bytes / (peak * 1e9) * 1e3
        line["prefill_phases"] = ph

    T2 = min(T, args.secondary_steps)

    def timed_decode_graph(steps_):
        """us per call of `steps_` decode steps x R replicas captured into a CUDA graph with the caches' current config."""
        with torch.cuda.stream(stream):
            stream.synchronize()
            g2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g2, stream=stream):
                for i in range(steps_):
                    for r, c in enumerate(caches):
                        c.decode_step(gq[i], gk[i], gv[i], victim_out=victims[r], stream=stream)
            g2.replay()
            a0, a1 = ev(), ev()
            a0.record(stream)
            g2.replay()
            g2.replay()
            a1.record(stream)
        torch.cuda.synchronize()
        return a0.elapsed_time(a1) * 1e3 / (2 * steps_ * R)

    if rank == 0 and not args.skip_decode_variants:
        from paper_2412_16187_b200 import HE_FLAG_EARLY_INPUTS, lib as he_lib
        import ctypes

        dv = {}
        # (a) the default order: q, k, v read only after the stream's previous kernel has ended
        for c in caches:
            c.cfg.flags &= ~HE_FLAG_EARLY_INPUTS
        us = timed_decode_graph(T2)
        dv["default_order"] = {"us_per_call": us, "frac": dec_bytes / us / 1e3 / peak,
                               "what": "HE_FLAG_EARLY_INPUTS off: the rows may come from the kernel enqueued just before the call"}
        for c in caches:
            c.cfg.flags |= HE_FLAG_EARLY_INPUTS if early else 0
        # (b) plain stream launches instead of a graph: the host enqueues every call (ctypes, addresses looked up once)
        L = he_lib()
        ptrs = [(ctypes.byref(c.cfg), ctypes.byref(c.ca), victims[r].data_ptr()) for r, c in enumerate(caches)]
        ins = [(gq[i].data_ptr(), gk[i].data_ptr(), gv[i].data_ptr()) for i in range(T2)]
        sp = stream.cuda_stream
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            for rep_ in range(2):
                if rep_ == 1:
                    torch.cuda.synchronize()
                    a0, a1 = ev(), ev()
                    t0 = time.perf_counter()
                    a0.record(stream)
                for q_, k_, v_ in ins:
                    for cf, ca_, vp_ in ptrs:
                        L.he_decode_step(cf, ca_, q_, k_, v_, vp_, None, None, sp)
            a1.record(stream)
            t_host = time.perf_counter() - t0
        torch.cuda.synchronize()
        dv["plain_launch"] = {"us_per_call": a0.elapsed_time(a1) * 1e3 / (T2 * R), "host_enqueue_us_per_call": 1e6 * t_host / (T2 * R),
                              "what": "the same calls as plain stream launches, enqueued one by one from the host"}
        # (c) one replica only: its 15 MB of tables, scores and slots stay in L2 between steps
        c0 = caches[0]
        with torch.cuda.stream(stream):
            stream.synchronize()
            g1 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g1, stream=stream):
                for i in range(T2):
                    c0.decode_step(gq[i], gk[i], gv[i], victim_out=victims[0], stream=stream)
            g1.replay()
            a0, a1 = ev(), ev()
            a0.record(stream)
            g1.replay()
            g1.replay()
            a1.record(stream)
        torch.cuda.synchronize()
        us = a0.elapsed_time(a1) * 1e3 / (2 * T2)
        dv["single_replica_l2_warm"] = {"us_per_call": us, "frac_of_hbm_peak": dec_bytes / us / 1e3 / peak,
                                        "what": "one cache stepped again and again: its working set stays in L2, so this is not an HBM figure"}
        line["decode_variants"] = dv
        del g1

    if rank == 0 and not args.skip_protected and w.n_sink == 0 and w.n_recent == 0:
        # ---- the paper's own setting (Section 4, configuration and setup): the first 4 and the newest 10 tokens stay
        for c in caches:
            c.cfg.n_sink, c.cfg.n_recent = 4, 10
        with torch.cuda.stream(stream):
            prefill_all()
            p0, p1 = ev(), ev()
            p0.record(stream)
            prefill_all()
            p1.record(stream)
        torch.cuda.synchronize()
        us = timed_decode_graph(T2)
        line["protected_4_10"] = {"n_sink": 4, "n_recent": 10, "prefill_ms_per_call": p0.elapsed_time(p1) / R,
                                  "decode_us_per_call": us, "decode_frac": dec_bytes / us / 1e3 / peak}
        for c in caches:
            c.cfg.n_sink, c.cfg.n_recent = 0, 0
        with torch.cuda.stream(stream):
            prefill_all()
        torch.cuda.synchronize()

    if rank == 0 and not args.skip_e2e:
        # ---- end to end: host buffers in, victims out, through he_decode_step_host_enqueue (copies inside the timed
        # region). Each step's q, k, v sit in one pinned block at the offsets the call recognises (one copy in), the
        # victims come back in one copy; addresses are looked up once, as a serving loop would.
        n_e2e = min(T, args.e2e_steps)
        esz = gq.element_size()
        qb, kb = gq[0].numel() * esz, gk[0].numel() * esz
        blk_bytes, (oq, ok_, ov) = caches[0].host_block_layout()
        blk = (blk_bytes + 255) // 256 * 256
        hblock = torch.empty((n_e2e, blk), dtype=torch.uint8).pin_memory()
        for i in range(n_e2e):
            hblock[i, oq:oq + qb] = gq[i].contiguous().view(torch.uint8).flatten().cpu()
            hblock[i, ok_:ok_ + kb] = gk[i].contiguous().view(torch.uint8).flatten().cpu()
            hblock[i, ov:ov + kb] = gv[i].contiguous().view(torch.uint8).flatten().cpu()
        # The layer replicas' calls of a step are independent, so they alternate between a few streams (each with its
        # own staging): the copies of one overlap the kernels and the copies of the others. A 0.79 MB host-to-device copy
        # costs 38 us back to back on one stream (20 GB/s; the link reaches 54 GB/s only from 16 MB per copy), so several
        # must be in flight: 1 / 2 / 4 / 8 streams gave 47 / 32 / 29 / 26 us per call. Every step ends with a synchronise, after
        # which that step's victims are readable on the host.
        hvic = torch.empty((R, B, H), dtype=torch.int32).pin_memory()
        e_streams = [torch.cuda.Stream() for _ in range(max(1, min(args.e2e_streams, R)))]
        ns = len(e_streams)
        stagings = [torch.empty(decode_staging_bytes(caches[0].cfg), dtype=torch.uint8, device="cuda") for _ in e_streams]
        base = hblock.data_ptr()
        calls = [(c, hvic[r].data_ptr(), stagings[r % ns].data_ptr(), stagings[r % ns].numel(), e_streams[r % ns].cuda_stream)
                 for r, c in enumerate(caches)]

        def e2e_step(i):
            qp = base + i * blk
            for c, op, sp_, sn, st_ in calls:
                c.decode_step_host_block_enqueue_raw(qp, op, sp_, sn, st_)
            for s_ in e_streams:
                s_.synchronize()
            return int(hvic[R - 1, 0, 0])  # the step's result is read on the host

        torch.cuda.synchronize()
        for i in range(3):
            e2e_step(i)
        t0 = time.perf_counter()
        for i in range(n_e2e):
            e2e_step(i)
        t_e2e = time.perf_counter() - t0
        line["e2e"] = {"value": units * n_e2e * R * world / t_e2e, "unit": UNIT, "h2d_bytes_per_step": qb + 2 * kb,
                       "d2h_bytes_per_step": hvic[0].numel() * 4, "us_per_call": 1e6 * t_e2e / (n_e2e * R),
                       "what": f"he_decode_step_host_block_enqueue, {n_e2e} decode steps x {R} layer replicas on {ns} alternating streams, "
                               "one synchronise and one host read of the victims per step; every call copies its pinned host "
                               "q/k/v block in (one copy) and its victims out inside the timed region"}

    if rank == 0 and not args.skip_folded and R > 1:
        # ---- secondary figure: the same decode kernel with all R replicas folded into ONE call (batch R*B), i.e. when
        # the per-call fixed costs (graph node, dependent load chain) are amortised over R times more units
        big = HashEvictCache(R * B, H, G, d, w.hash_bits, np.tile(budgets, R), torch.from_numpy(wl.gen_W(w)), dtype=tdt,
                             n_sink=w.n_sink, n_recent=w.n_recent, write_scores=True, packed_codes=args.packed_codes,
                             early_inputs=not args.no_early_inputs)
        for r, c in enumerate(caches):
            sl = slice(r * B, (r + 1) * B)
            big.codes_storage[sl].copy_(c.codes_storage)
            big.pos[sl].copy_(c.pos)
            big.fill[sl].copy_(c.fill)
            big.next_pos[sl].copy_(c.next_pos)
        nf = min(T, 8)
        fq, fk, fv = (x[:nf].repeat(1, R, 1, 1).contiguous() for x in (gq, gk, gv))
        fvic = torch.empty((R * B, H), dtype=torch.int32, device="cuda")
        with torch.cuda.stream(stream):
            for i in range(3):
                big.decode_step(fq[i], fk[i], fv[i], victim_out=fvic, stream=stream)
            f0, f1 = ev(), ev()
            f0.record(stream)
            for rep in range(4):
                for i in range(nf):
                    big.decode_step(fq[i], fk[i], fv[i], victim_out=fvic, stream=stream)
            f1.record(stream)
        torch.cuda.synchronize()
        us = f0.elapsed_time(f1) * 1e3 / (4 * nf)
        fbytes = decode_bytes_per_call(w.scaled(batch=R * w.batch), np.tile(budgets, R))
        line["decode_folded"] = {"what": f"one he_decode_step over {R * B} sequences ({R} replicas folded into the batch)",
                                 "us_per_call": us, "evictions_per_s": R * units / (us * 1e-6),
                                 "achieved_gbs": fbytes / us / 1e3, "frac": fbytes / us / 1e3 / peak}
        del big

    if rank == 0 and not args.skip_attend:
        # ---- secondary figure: Eq. 1 over the compressed caches the steps above left behind (Algorithm 1 line 6),
        # one he_attend call per layer replica, rotating over the replicas so that K/V come from HBM, not L2
        aq = gq[T - 1]
        aout = torch.empty((B, H * G, d), dtype=torch.float32, device="cuda")
        reps = max(1, int(np.ceil(64 / R)))
        with torch.cuda.stream(stream):
            for c in caches[:3]:
                c.attend(aq, aout, stream=stream)
            a0, a1 = ev(), ev()
            a0.record(stream)
            for _ in range(reps):
                for c in caches:
                    c.attend(aq, aout, stream=stream)
            a1.record(stream)
        torch.cuda.synchronize()
        us = a0.elapsed_time(a1) * 1e3 / (reps * R)
        esz = 2 if w.dtype == "bf16" else 4
        abytes = float(caches[0].fill.sum().item()) * 2 * d * esz + B * H * G * d * (esz + 4)
        line["attend"] = {"what": "he_attend: softmax(q K^T / sqrt(d)) V over the valid slots of every unit, one call per replica",
                          "us_per_call": us, "bound": "hbm", "achieved": abytes / us / 1e3, "peak": peak, "unit": "GB/s",
                          "frac": abytes / us / 1e3 / peak, "algorithmic_bytes_per_call": abytes,
                          "kv_bytes_all_replicas": abytes * R}

    if rank == 0 and not args.skip_oneshot:
        # ---- secondary figure: the one-shot ranking of Appendix C as a prompt-compression variant (not Section 3's
        # procedure): same inputs, every prompt query hashed, linear-time ranking, same gather. Runs last: it
        # overwrites the caches.
        with torch.cuda.stream(stream):
            for c in caches:  # untimed: every cache allocates its ranking workspace on its first call
                c.prefill_oneshot(dQ, dK, dV, dplen, Nmax, stream=stream)
            stream.synchronize()
            o0, o1 = ev(), ev()
            o0.record(stream)
            for c in caches:
                c.prefill_oneshot(dQ, dK, dV, dplen, Nmax, stream=stream)
            o1.record(stream)
        torch.cuda.synchronize()
        ms = o0.elapsed_time(o1) / R
        esz = 2 if w.dtype == "bf16" else 4
        obytes = float(plens.sum()) * H * (1 + G) * d * esz + float(np.minimum(plens, budgets).sum()) * H * 4 * d * esz
        line["prefill_oneshot"] = {"what": "he_prefill_oneshot: averaged-Hamming ranking (Appendix C), one call per replica",
                                   "ms_per_call": ms, "keys_per_s": float(plens.sum()) * H / (ms * 1e-3), "bound": "hbm",
                                   "achieved": obytes / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                                   "frac": obytes / (ms * 1e-3) / 1e9 / peak, "algorithmic_bytes_per_call": obytes}

    if rank == 0 and not args.skip_oneshot:
        # ---- secondary figure: attention loss (Section 4.6) of the three prompt-compression policies on this synthetic
        # workload: mass of softmax(q K^T / sqrt(d)) over the whole prompt that falls on tokens no longer cached, for
        # the first decode query of every head. Synthetic keys and queries: the numbers say nothing about a real model.
        c0 = caches[0]
        lo = torch.empty((B, H * G), dtype=torch.float32, device="cuda")
        losses = {}
        with torch.cuda.stream(stream):
            for name, fill in (("algorithm_1", lambda: c0.prefill_compress(dQ, dK, dV, dplen, Nmax, workspace=ws, stream=stream)),
                               ("oneshot_avg_hamming", lambda: c0.prefill_oneshot(dQ, dK, dV, dplen, Nmax, stream=stream)),
                               ("l2_norm", lambda: c0.prefill_oneshot_l2(dK, dV, dplen, Nmax, stream=stream))):
                fill()
                c0.attention_loss(gq[0], dK, out=lo, stream=stream)
                stream.synchronize()
                losses[name] = float(lo.mean().item())
            l0, l1, l2 = ev(), ev(), ev()
            l0.record(stream)
            for _ in range(4):
                c0.attention_loss(gq[0], dK, out=lo, stream=stream)
            l1.record(stream)
            for _ in range(4):
                c0.prefill_oneshot_l2(dK, dV, dplen, Nmax, stream=stream)
            l2.record(stream)
        torch.cuda.synchronize()
        ms = l0.elapsed_time(l1) / 4
        line["prefill_oneshot_l2"] = {"what": "he_prefill_oneshot_l2: keep the lowest key norms (comparison policy), per call",
                                      "ms_per_call": l1.elapsed_time(l2) / 4,
                                      "keys_per_s": float(plens.sum()) * H / (l1.elapsed_time(l2) / 4 * 1e-3)}
        esz = 2 if w.dtype == "bf16" else 4
        lbytes = float(plens.sum()) * H * d * esz
        line["attention_loss"] = {"what": "he_attention_loss after each prompt-compression policy (mean over heads), synthetic data",
                                  "mean_loss": losses, "ms_per_call": ms, "achieved_gbs": lbytes / (ms * 1e-3) / 1e9,
                                  "frac": lbytes / (ms * 1e-3) / 1e9 / peak}

    if rank == 0 and not args.skip_largest_prefill and w.name == "throughput_batch":
        # ---- he_prefill_compress on the configuration that is largest for prefill: long_prefill, its 32 layers folded
        # into the batch (256 units, 32768-token prompts, 9830 slots). Layer 0's q/k/v are generated on the host by the
        # seeded generator; the other 31 layers are that layer's tokens rotated by a layer-dependent offset on the
        # device (same distribution, different order, own memory: 12.9 GB), which keeps the set-up to seconds.
        w4 = wl.CONFIGS["long_prefill"]
        B4, N4 = w4.n_seq, w4.max_prompt_len
        k0, v0, q0 = (up(wl.gen_tokens(w4, x, 0, 1, 0, N4)[0]) for x in "kvq")
        dK4 = torch.empty((B4, H, N4, d), dtype=tdt, device="cuda")
        dV4 = torch.empty_like(dK4)
        dQ4 = torch.empty((B4, w4.n_kv_heads * w4.group_size, N4, d), dtype=tdt, device="cuda")
        for l in range(B4):
            dK4[l], dV4[l], dQ4[l] = (torch.roll(x, shifts=l * 997, dims=1) for x in (k0, v0, q0))
        b4, p4 = w4.budgets(), w4.prompt_lens()
        c4 = HashEvictCache(B4, w4.n_kv_heads, w4.group_size, d, w4.hash_bits, b4, torch.from_numpy(wl.gen_W(w4)), dtype=tdt)
        ws4 = c4.workspace(N4)
        dp4 = torch.from_numpy(p4).cuda()
        with torch.cuda.stream(stream):
            c4.prefill_compress(dQ4, dK4, dV4, dp4, N4, workspace=ws4, stream=stream)
        torch.cuda.synchronize()
        ph4 = phase_split([c4], dQ4, dK4, dV4, dp4, N4, ws4, reps=3)
        bytes4 = prefill_bytes_per_call(w4, b4, p4)
        ph4["replay_bound"] = replay_bound_obj(w4, b4, p4, ph4["schedule_replay_ms"])
        ph4["replay_bound"]["hbm_floor_ms_of_the_whole_call"] = bytes4 / (peak * 1e9) * 1e3
        gbs4 = bytes4 / (ph4["call_ms"] * 1e-3) / 1e9
        line["prefill_largest"] = {"workload": "long_prefill, 32 layers folded into the batch (256 units, N = 32768, C = 9830)",
                                   "ms_per_call": ph4["call_ms"], "keys_per_s": float(p4.sum()) * w4.n_kv_heads / (ph4["call_ms"] * 1e-3),
                                   "bound": "hbm", "achieved": gbs4, "peak": peak, "unit": "GB/s", "frac": gbs4 / peak,
                                   "frac_of_nominal_8TBs": gbs4 / NOMINAL_HBM_GBS, "algorithmic_bytes_per_call": bytes4,
                                   "phases": ph4,
                                   "data": "layer 0 from the seeded generator, layers 1..31 = layer 0 with its tokens rotated by 997 * layer"}
        del dK4, dV4, dQ4, c4, ws4, k0, v0, q0

    if rank == 0:
        line["clocks"] = clocks
        if not args.skip_cpu_baseline and world == 1:
            threads = len(os.sched_getaffinity(0))
            r = oracle_sample(w, args.ref_seqs, args.ref_decode_steps, threads)
            line["cpu_baseline"] = {"value": r["evictions_per_s"], "unit": UNIT, "cores": threads, "kind": "oracle",
                                    "sample": r["sample"], "prefill_keys_per_s": r["prefill_keys_per_s"],
                                    "seconds": r["t_prefill_s"] + r["t_decode_s"]}
            r1 = oracle_sample(w, 1, min(32, args.ref_decode_steps), 1)
            line["cpu_baseline"].update(value_1_thread=r1["evictions_per_s"], prefill_keys_per_s_1_thread=r1["prefill_keys_per_s"],
                                        sample_1_thread=r1["sample"], seconds_1_thread=r1["t_prefill_s"] + r1["t_decode_s"])
        line["wall_s_timed_region"] = t_wall
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="throughput_batch", choices=list(wl.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--replicas", type=int, default=None, help="independent layer replicas cycled by the decode loop")
    ap.add_argument("--decode-steps", type=int, default=None)
    ap.add_argument("--hash-bits", type=int, default=None, help="override b (hash-dimension sweep of Section 4.7)")
    ap.add_argument("--packed-codes", action="store_true",
                    help="code table with ceil(b/8) bytes per slot (HE_FLAG_PACKED_CODES) instead of 32-bit words")
    ap.add_argument("--batch", type=int, default=None, help="fewer sequences (profiling captures on a small case)")
    ap.add_argument("--prompt-factor", type=int, default=None, help="ragged workloads: prompt = factor x budget")
    ap.add_argument("--no-graph", action="store_true", help="plain stream launches instead of a CUDA graph")
    ap.add_argument("--no-early-inputs", action="store_true",
                    help="leave HE_FLAG_EARLY_INPUTS off (q, k, v are then read only after the stream's previous kernel has ended)")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-phases", action="store_true", help="skip the per-phase split of he_prefill_compress")
    ap.add_argument("--skip-decode-variants", action="store_true", help="skip default-order / plain-launch / one-replica decode figures")
    ap.add_argument("--skip-protected", action="store_true", help="skip the figures with the paper's protected windows (4, 10)")
    ap.add_argument("--skip-largest-prefill", action="store_true", help="skip he_prefill_compress on long_prefill (32 layers folded)")
    ap.add_argument("--secondary-steps", type=int, default=128, help="decode steps of the secondary decode figures")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-oneshot", action="store_true", help="skip the he_prefill_oneshot figure")
    ap.add_argument("--skip-attend", action="store_true", help="skip the he_attend figure")
    ap.add_argument("--skip-folded", action="store_true", help="skip the secondary all-replicas-in-one-call decode figure")
    ap.add_argument("--e2e-steps", type=int, default=64)
    ap.add_argument("--e2e-streams", type=int, default=8, help="streams the layer replicas' end-to-end calls alternate between")
    ap.add_argument("--ref-seqs", type=int, default=12, help="sequences in the oracle's bounded sample")
    ap.add_argument("--ref-decode-steps", type=int, default=128)
    args = ap.parse_args()
    global PACKED_CODES
    PACKED_CODES = args.packed_codes
    w = wl.CONFIGS[args.workload]
    if args.decode_steps is not None:
        w = w.scaled(decode_steps=args.decode_steps)
    if args.hash_bits is not None:
        w = w.scaled(hash_bits=args.hash_bits)
    if args.batch is not None:
        w = w.scaled(batch=args.batch)
    if args.prompt_factor is not None:
        w = w.scaled(prompt_factor=args.prompt_factor)
    if args.replicas is None:
        args.replicas = DEFAULT_REPLICAS[args.workload]
    if args.warmup < 3 and args.impl == "ours":
        print("note: fewer than 3 warm-up steps", file=sys.stderr)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
