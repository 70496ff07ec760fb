"""Full-size cross-check of the replay implementations: at the full workload sizes the oracle follows sampled units
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


RANDOM_SCRIPT = r"""
import sys, json, hashlib, numpy as np, torch
sys.path.insert(0, %r)
from paper_2412_16187_b200 import HashEvictCache, device_error_count
rng = np.random.default_rng(2024)
out = []
for trial in range(24):
    B = int(rng.integers(1, 5)); H = int(rng.integers(1, 5)); G = int(rng.choice([1, 2, 3, 4, 5, 7, 8])); d = 128
    b = int(rng.choice([4, 8, 13, 16, 24, 32, 33, 40, 64]))
    cmax = int(rng.choice([130, 300, 700, 1500, 3000, 4096, 4500, 6000]))
    budgets = rng.integers(max(40, cmax // 3), cmax + 1, size=B).astype(np.int32)
    N = int(rng.integers(cmax // 2, 3 * cmax))
    plens = rng.integers(0, N + 1, size=B).astype(np.int32); plens[0] = N
    prot = rng.random() < 0.5
    n_sink = int(rng.integers(0, 6)) if prot else 0
    n_recent = int(rng.integers(0, 30)) if prot else 0
    g = torch.Generator(device="cuda"); g.manual_seed(trial)
    K = torch.randn(B, H, N, d, device="cuda", generator=g)
    if rng.random() < 0.3:  # little variety in the keys: many equal distances
        K = K[:, :, :1, :] + 0.05 * K
    Q = torch.randn(B, H * G, N, d, device="cuda", generator=g)
    K = K.to(torch.bfloat16); Q = Q.to(torch.bfloat16)
    c = HashEvictCache(B, H, G, d, b, budgets, torch.randn(d, b, device="cuda", generator=g), dtype=torch.bfloat16,
                       n_sink=n_sink, n_recent=n_recent)
    c.prefill_compress(Q, K, K, torch.from_numpy(plens).cuda())
    torch.cuda.synchronize()
    h = hashlib.sha256()
    for t in (c.codes, c.pos, c.scores, c.fill, c.next_pos):
        h.update(t.cpu().numpy().tobytes())
    out.append(h.hexdigest())
assert device_error_count() == 0
print("DIGESTS " + json.dumps(out))
""" % (ROOT,)


def test_replay_implementations_agree_on_random_shapes():
    """Random group sizes (1..8), code widths (4..64, odd ones included), ragged budgets from 40 to 6000 slots, ragged
    prompt lengths (empty and shorter than the budget included), protected windows, keys with little variety."""
    def digests(env):
        e = dict(os.environ, **env)
        r = subprocess.run([sys.executable, "-c", RANDOM_SCRIPT], env=e, capture_output=True, text=True, timeout=900)
        assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
        return json.loads([l for l in r.stdout.splitlines() if l.startswith("DIGESTS ")][-1][len("DIGESTS "):])

    ref = digests({"HE_TC_REPLAY": "0"})
    assert digests({"HE_TC_REPLAY": "1"}) == ref
    assert digests({"HE_TC_REPLAY": "1", "HE_TC_REPLAY_BF16": "1"}) == ref
