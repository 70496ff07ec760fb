"""HE_FLAG_EARLY_INPUTS: the decode kernel that hashes the step's rows before it waits for the stream's previous
kernel. It must give the results of the default kernel: against the oracle step by step, and when many calls are
enqueued back to back (same cache step after step, and several caches in turn) with no synchronise in between."""
import numpy as np
import pytest
import torch

from cases import PARITY_CASES
from paper_2412_16187_b200 import workloads as wl
from parity import Case, to_dev

pytestmark = pytest.mark.gpu

STATE = ("codes", "pos", "fill", "next_pos", "scores", "k_cache", "v_cache")


@pytest.mark.parametrize("name", ["tiny", "llama2_7b_layer", "llama3_8b_gqa", "throughput_batch", "protected_gqa", "long_prefill"])
def test_early_inputs_decode_matches_oracle(name):
    w = PARITY_CASES[name]
    case = Case(w, early_inputs=True)
    flips, fragile = case.prefill()
    case.compare_state()
    f2, g2 = case.decode(min(w.decode_steps, 24), check_every=6)
    assert flips + f2 <= fragile + g2


def test_early_inputs_generic_group_size_and_odd_bits():
    w = PARITY_CASES["protected_gqa"].scaled(group_size=7, hash_bits=40, batch=2, prompt_len=300, budget=97, decode_steps=12)
    case = Case(w, early_inputs=True)
    case.prefill()
    case.decode(12)


def test_early_inputs_decode_from_empty_cache():
    """Appending steps (nothing scored) and the first evictions, fp32 rows."""
    w = PARITY_CASES["tiny"].scaled(n_sink=1, n_recent=2)
    a, b = Case(w), Case(w, early_inputs=True)
    a.prefill()
    b.gpu.reset()
    rows = [(b.dQ[:, :, t].contiguous(), b.dK[:, :, t].contiguous(), b.dV[:, :, t].contiguous()) for t in range(w.prompt_len)]
    torch.cuda.synchronize()
    for q, k, v in rows:
        b.gpu.decode_step(q, k, v)
    torch.cuda.synchronize()
    for name in STATE:
        assert torch.equal(getattr(a.gpu, name), getattr(b.gpu, name)), name


@pytest.mark.parametrize("name", ["throughput_batch", "llama3_8b_gqa"])
def test_back_to_back_calls_give_the_same_state_with_and_without_the_flag(name):
    """T steps x 3 caches enqueued on one stream without any synchronise (inputs staged beforehand, as the flag
    requires): every call overlaps its predecessor, yet each cache must end exactly where the default kernel,
    synchronised after every call, leaves it. Also replayed from a CUDA graph."""
    w = PARITY_CASES[name]
    T = 40
    dq, dk, dv = (to_dev(wl.gen_decode_inputs(w, x, 0, T), w) for x in "qkv")
    ref = Case(w)
    ref.prefill()
    want_vic = []
    for i in range(T):
        want_vic.append(ref.gpu.decode_step(dq[i], dk[i], dv[i]).clone())
        torch.cuda.synchronize()
    caches = [Case(w, early_inputs=True) for _ in range(3)]
    for c in caches:
        c.gpu.prefill_compress(c.dQ, c.dK, c.dV, c.dplen)
    vic = torch.empty((3, T, w.n_seq, w.n_kv_heads), dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(T // 2):
            for ci, c in enumerate(caches):
                c.gpu.decode_step(dq[i], dk[i], dv[i], victim_out=vic[ci, i], stream=stream)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(T // 2, T):
                for ci, c in enumerate(caches):
                    c.gpu.decode_step(dq[i], dk[i], dv[i], victim_out=vic[ci, i], stream=stream)
        graph.replay()
    torch.cuda.synchronize()
    for ci, c in enumerate(caches):
        for i in range(T):
            assert torch.equal(vic[ci, i], want_vic[i]), (ci, i)
        for n in STATE:
            assert torch.equal(getattr(ref.gpu, n), getattr(c.gpu, n)), n
