"""The three implementations of Eq. 2 on the device (CUDA-core kernel, tensor-core kernel fed by TMA, tensor-core
kernel fed by cp.async) against the oracle, each forced through environment switches in a fresh process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SCRIPT = r"""
import sys, numpy as np, torch
sys.path.insert(0, %r); sys.path.insert(0, %r)
from paper_2412_16187_b200 import hash_keys, device_error_count, workloads as wl
from parity import check_hash_stage, codes_np, to_dev
for (d, b, rows) in [(128, 64, 9000), (128, 16, 8200), (64, 33, 8192 + 5)]:
    w = wl.Workload("h", 23, 1, 1, 1, 1, d, "bf16", b, rows, 4, 0, wl.KIND_DRIFT)
    W = wl.gen_W(w); x = wl.gen_tokens(w, "k", 0, 1, 0, rows)[0, 0]
    got = codes_np(hash_keys(to_dev(x, w), torch.from_numpy(W).cuda()))
    flips, fragile = check_hash_stage(x, W, "bf16", got)
    assert flips <= fragile
assert device_error_count() == 0
print("ok")
""" % (ROOT, os.path.join(ROOT, "tests"))


@pytest.mark.parametrize("env", [{}, {"HE_DISABLE_TMA": "1"}, {"HE_DISABLE_TC": "1"}], ids=["tc_tma", "tc_cp_async", "cuda_cores"])
def test_hash_path(env):
    e = dict(os.environ, **env)
    r = subprocess.run([sys.executable, "-c", SCRIPT], env=e, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "ok" in r.stdout, r.stdout + r.stderr
