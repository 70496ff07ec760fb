"""Writes tests/golden/digests.json from the CPU oracle alone (never from the CUDA path).

Run from the repository root:  python tests/golden/make_digests.py
A digest is the 64-bit FNV-1a hash of an array's bytes. They freeze the oracle's behaviour on the
seeded parity cases so that a later edit of the oracle cannot drift unnoticed; the GPU results are
always compared with the oracle's full arrays, not with these digests.
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle  # noqa: E402
from cases import PARITY_CASES  # noqa: E402
from paper_2412_16187_b200 import workloads as wl  # noqa: E402

DIGEST_CASES = ("tiny", "protected_tiny", "throughput_batch")


def fnv1a64(a: np.ndarray) -> str:
    h = 0xCBF29CE484222325
    for byte in np.ascontiguousarray(a).tobytes():
        h = ((h ^ byte) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return f"{h:016x}"


def run_case(w):
    """Prefill then all decode steps in the oracle; returns the arrays that are digested."""
    Nmax = w.max_prompt_len
    W = wl.gen_W(w)
    K = wl.gen_tokens(w, "k", 0, w.n_seq, 0, Nmax)
    Q = wl.gen_tokens(w, "q", 0, w.n_seq, 0, Nmax)
    V = wl.gen_tokens(w, "v", 0, w.n_seq, 0, Nmax)
    oc = oracle.OracleCache(w.n_seq, w.n_kv_heads, w.group_size, w.head_dim, w.hash_bits, w.max_budget, w.budgets(),
                            w.dtype, n_sink=w.n_sink, n_recent=w.n_recent, threads=os.cpu_count() or 1)
    kc, _ = oc.prefill(W, Q, K, V, w.prompt_lens(), want_codes=True)
    pos_after_prefill = oc.pos.copy()
    dq = wl.gen_decode_inputs(w, "q", 0, w.decode_steps)
    dk = wl.gen_decode_inputs(w, "k", 0, w.decode_steps)
    dv = wl.gen_decode_inputs(w, "v", 0, w.decode_steps)
    victims = np.stack([oc.step(W, dq[i], dk[i], dv[i])[0] for i in range(w.decode_steps)])
    return {"prompt_key_codes": kc, "pos_after_prefill": pos_after_prefill, "decode_victims": victims,
            "final_pos": oc.pos, "final_codes": oc.codes, "final_scores": oc.scores}


def main():
    out = {name: {k: fnv1a64(v) for k, v in run_case(PARITY_CASES[name]).items()} for name in DIGEST_CASES}
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "digests.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
