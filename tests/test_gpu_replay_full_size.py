"""Full-size cross-check of the replay implementations: at BASELINE sizes the oracle can only follow sampled units
(tests/test_gpu_parity.py does that), so here the tensor-core replay (8-bit and bf16 operands) and the CUDA-core
replay, each of which is checked against the oracle on smaller shapes, must leave bit-identical caches on the whole
throughput_batch workload (also with the paper's protected windows) and on four layers of long_prefill (9830-slot
budgets, tables in global memory)."""
import hashlib
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SCRIPT = r"""
import sys, json, hashlib, numpy as np, torch
sys.path.insert(0, %r)
from paper_2412_16187_b200 import HashEvictCache, device_error_count, workloads as wl
out = {}
for name, w in (("throughput_batch", wl.CONFIGS["throughput_batch"]), ("long_prefill", wl.CONFIGS["long_prefill"].scaled(layers=4)),
                ("throughput_batch_protected", wl.CONFIGS["throughput_batch"].scaled(batch=32, n_sink=4, n_recent=10)),
                ("long_prefill_protected", wl.CONFIGS["long_prefill"].scaled(layers=2, n_sink=4, n_recent=10))):
    B, H, G, d = w.n_seq, w.n_kv_heads, w.group_size, w.head_dim
    plens, Nmax = w.prompt_lens(), w.max_prompt_len
    def up(a):
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    dK = torch.zeros((B, H, Nmax, d), dtype=torch.bfloat16, device="cuda"); dV = torch.zeros_like(dK)
    dQ = torch.zeros((B, H * G, Nmax, d), dtype=torch.bfloat16, device="cuda")
    for s in range(B):
        n = int(plens[s])
        dK[s, :, :n] = up(wl.gen_tokens(w, "k", s, 1, 0, n)[0]); dV[s, :, :n] = up(wl.gen_tokens(w, "v", s, 1, 0, n)[0])
        dQ[s, :, :n] = up(wl.gen_tokens(w, "q", s, 1, 0, n)[0])
    c = HashEvictCache(B, H, G, d, w.hash_bits, w.budgets(), torch.from_numpy(wl.gen_W(w)), dtype=torch.bfloat16, n_sink=w.n_sink,
                       n_recent=w.n_recent)
    c.prefill_compress(dQ, dK, dV, torch.from_numpy(plens).cuda())
    torch.cuda.synchronize()
    h = hashlib.sha256()
    for t in (c.codes, c.pos, c.scores, c.fill, c.next_pos, c.k_cache.view(torch.int16), c.v_cache.view(torch.int16)):
        h.update(t.cpu().numpy().tobytes())
    out[name] = h.hexdigest()
    del dK, dV, dQ, c
    torch.cuda.empty_cache()
assert device_error_count() == 0
print("DIGESTS " + json.dumps(out))
""" % (ROOT,)


def run(env):
    e = dict(os.environ, **env)
    r = subprocess.run([sys.executable, "-c", SCRIPT], env=e, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("DIGESTS ")][-1]
    return json.loads(line[len("DIGESTS "):])


def test_replay_implementations_agree_at_full_size():
    ref = run({"HE_TC_REPLAY": "0"})
    assert run({"HE_TC_REPLAY": "1"}) == ref
    assert run({"HE_TC_REPLAY": "1", "HE_TC_REPLAY_BF16": "1"}) == ref
