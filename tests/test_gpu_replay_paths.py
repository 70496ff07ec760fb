"""The implementations of the prompt replay (tensor-core kernel with 8-bit or bf16 operands, CUDA-core kernels)
against the oracle, each forced through the environment switches in a fresh process, on shapes that cover one-word and two-word codes, group
sizes 1, 3 and 4, budgets that are not multiples of the 128-slot tile, ragged budgets, prompts that end inside a
128-step block, prompts shorter than the budget, protected windows, and keys with little variety (many equal distances, so the
lowest-slot rule and the repair of stale tile maxima are exercised)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SCRIPT = r"""
import sys, numpy as np, torch
sys.path.insert(0, %r); sys.path.insert(0, %r)
from paper_2412_16187_b200 import device_error_count, workloads as wl
from cases import PARITY_CASES
from parity import Case
C = wl.CONFIGS
shapes = [
    PARITY_CASES["tiny"],
    PARITY_CASES["llama2_7b_layer"].scaled(prompt_len=1300, budget=777, decode_steps=2),
    PARITY_CASES["llama3_8b_gqa"].scaled(batch=2, prompt_len=1500, budget=1000, decode_steps=2),
    PARITY_CASES["throughput_batch"].scaled(batch=4, decode_steps=2),
    C["throughput_batch"].scaled(batch=2, budget_lo=130, budget_hi=300, group_size=3, hash_bits=40, decode_steps=2),
    C["llama3_8b_gqa"].scaled(batch=1, prompt_len=640, budget=129, hash_bits=4, decode_steps=2),
    C["llama3_8b_gqa"].scaled(batch=1, prompt_len=2100, budget=2049, hash_bits=8, decode_steps=2),
    # the paper's protected windows (first 4, newest 10), also with few-bit codes whose ties favour the sink slots, a window
    # longer than a quarter of a block, and sinks without a recent window
    PARITY_CASES["protected_gqa"].scaled(decode_steps=2),
    PARITY_CASES["protected_tiny"].scaled(decode_steps=2),
    C["llama3_8b_gqa"].scaled(batch=2, prompt_len=1500, budget=700, decode_steps=2, n_sink=4, n_recent=10),
    C["llama3_8b_gqa"].scaled(batch=1, prompt_len=900, budget=260, hash_bits=4, decode_steps=2, n_sink=4, n_recent=10),
    C["throughput_batch"].scaled(batch=2, budget_lo=200, budget_hi=400, decode_steps=2, n_sink=2, n_recent=45),
    C["llama2_7b_layer"].scaled(prompt_len=700, budget=300, decode_steps=2, n_sink=7, n_recent=0),
    # budgets above 4096 slots (tables in global memory), plain and with protected windows up to the 32-token ring
    C["long_prefill"].scaled(layers=1, n_kv_heads=2, prompt_len=7000, budget=4500, decode_steps=2),
    C["long_prefill"].scaled(layers=1, n_kv_heads=2, prompt_len=7000, budget=4500, decode_steps=2, n_sink=4, n_recent=10),
    C["long_prefill"].scaled(layers=1, n_kv_heads=1, prompt_len=6000, budget=4200, hash_bits=8, decode_steps=2, n_sink=3, n_recent=32),
    # four-bit codes over several tiles: most steps hit a stale tile maximum, so blocks are cut short after 64 repairs
    C["llama3_8b_gqa"].scaled(batch=1, prompt_len=1800, budget=700, hash_bits=4, decode_steps=2),
]
for w in shapes:
    case = Case(w)
    case.prefill()
    case.compare_state()
    case.decode(2)
# short and empty prompts next to evicting ones
w = PARITY_CASES["throughput_batch"].scaled(batch=4, decode_steps=2)
case = Case(w)
b = w.budgets()
case.plen = np.array([0, 5, int(b[2]), int(b[3]) + 1], dtype=np.int32)
case.dplen = torch.from_numpy(case.plen).cuda()
case.prefill()
case.compare_state()
assert device_error_count() == 0
print("ok")
""" % (ROOT, os.path.join(ROOT, "tests"))


@pytest.mark.parametrize("env", [{"HE_TC_REPLAY": "1"}, {"HE_TC_REPLAY": "1", "HE_TC_REPLAY_BF16": "1"}, {"HE_TC_REPLAY": "0"}],
                         ids=["tensor_cores_fp8", "tensor_cores_bf16", "cuda_cores"])
def test_replay_path(env):
    e = dict(os.environ, **env)
    r = subprocess.run([sys.executable, "-c", SCRIPT], env=e, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
