"""Device-side inputs the host cannot see, the two roundings of Eq. 2, and the bounds-checking build."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from cases import PARITY_CASES
from paper_2412_16187_b200 import HashEvictCache, hash_keys
from paper_2412_16187_b200 import workloads as wl
from parity import Case, check_hash_stage, codes_np, to_dev, torch_dtype

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
STATE = ("codes", "pos", "fill", "next_pos", "scores", "k_cache", "v_cache")


def test_prompt_lengths_beyond_the_maximum_are_clamped():
    """prompt_len lives on the device; a value above max_prompt_len counts as max_prompt_len and a negative one as 0
    (the prompt-code scratch holds max_prompt_len rows per unit), for every replay kernel."""
    for name in ("throughput_batch", "llama3_8b_gqa", "tiny"):
        w = PARITY_CASES[name].scaled(decode_steps=0)
        good, bad = Case(w), Case(w)
        Nmax = w.max_prompt_len
        want = good.plen.copy()
        want[0] = Nmax
        wild = want.copy()
        wild[0] = Nmax + 1000
        if w.n_seq > 1:
            want[1] = 0
            wild[1] = -7
        good.plen, good.dplen = want, torch.from_numpy(want).cuda()
        good.prefill()
        good.compare_state()
        bad.gpu.prefill_compress(bad.dQ, bad.dK, bad.dV, torch.from_numpy(wild).cuda(), Nmax)
        torch.cuda.synchronize()
        for n in STATE:
            assert torch.equal(getattr(good.gpu, n), getattr(bad.gpu, n)), (name, n)


@pytest.mark.parametrize("early", [False, True])
def test_a_budget_below_one_on_the_device_stores_nothing(early):
    """Without a host mirror the host cannot reject the budget; the kernels must not turn it into a wild slot index."""
    w = PARITY_CASES["llama3_8b_gqa"].scaled(batch=3, prompt_len=300, budget=64, decode_steps=2)
    W = torch.from_numpy(wl.gen_W(w))
    c = HashEvictCache(3, w.n_kv_heads, w.group_size, w.head_dim, w.hash_bits, [64, 64, 64], W, dtype=torch.bfloat16,
                       host_budget_mirror=False, early_inputs=early)
    c.budget.copy_(torch.tensor([64, 0, -5], dtype=torch.int32))
    case = Case(w.scaled(batch=3))
    c.prefill_compress(case.dQ, case.dK, case.dV, case.dplen)
    torch.cuda.synchronize()
    assert c.fill.cpu().tolist() == [[64] * w.n_kv_heads, [0] * w.n_kv_heads, [0] * w.n_kv_heads]
    before = {n: getattr(c, n)[1:].clone() for n in STATE}
    dq, dk, dv = (to_dev(wl.gen_decode_inputs(w.scaled(batch=3), x, 0, 2), w) for x in "qkv")
    for i in range(2):
        vic = c.decode_step(dq[i], dk[i], dv[i])
        torch.cuda.synchronize()
        assert (vic[1:] == -1).all() and (vic[0] >= 0).all() and (vic[0] < 64).all()
    for n in STATE:
        assert torch.equal(getattr(c, n)[1:], before[n]), n


def test_the_two_roundings_of_eq2_agree_outside_the_fragile_bits():
    """The same bf16 rows through the bulk tensor-core projection (he_hash_keys), the per-unit decode kernel (CUDA
    cores) and the decode kernel of HE_FLAG_EARLY_INPUTS (warp-level tensor-core instructions): each may differ from
    the oracle, and hence from the others, only in bits whose fp64 projection is within the Eq. 2 tolerance of zero."""
    w = wl.CONFIGS["throughput_batch"].scaled(budget_lo=8, budget_hi=8, prompt_factor=1, decode_steps=4)
    W = wl.gen_W(w)
    dq, dk, dv = (wl.gen_decode_inputs(w, x, 0, 4) for x in "qkv")
    gq, gk, gv = (to_dev(x, w) for x in (dq, dk, dv))
    rows = dq.reshape(-1, w.head_dim)
    assert rows.shape[0] >= 8192  # enough 128-row tiles for he_hash_keys to take its tensor-core kernel
    ref, fragile = oracle.hash_rows(np.ascontiguousarray(rows), W, w.dtype, want_fragile=True)
    got = {"bulk": codes_np(hash_keys(to_dev(rows, w), torch.from_numpy(W).cuda())).reshape(ref.shape)}
    for name, early in (("decode", False), ("decode_early", True)):
        c = HashEvictCache(w.n_seq, w.n_kv_heads, w.group_size, w.head_dim, w.hash_bits, w.budgets(), torch.from_numpy(W),
                           dtype=torch.bfloat16, early_inputs=early)
        qc = torch.empty((w.n_seq, w.n_kv_heads * w.group_size, c.Wd), dtype=torch.int32, device="cuda")
        out = []
        for i in range(4):
            c.decode_step(gq[i], gk[i], gv[i], qcodes_out=qc)
            torch.cuda.synchronize()
            out.append(codes_np(qc).copy())
        got[name] = np.stack(out).reshape(ref.shape)
    for name, g in got.items():
        bad = (g ^ ref) & ~fragile
        assert not bad.any(), f"{name}: {int(np.count_nonzero(bad))} code words differ from the oracle outside the fragile set"
    for a in got:
        for b in got:
            assert not ((got[a] ^ got[b]) & ~fragile).any(), (a, b)


def test_bf16_decode_from_an_empty_cache_matches_prefill_up_to_fragile_bits():
    """he_reset + N x he_decode_step against he_prefill_compress on bf16 rows, where the prompt is hashed in bulk on
    tensor cores and the steps' rows inside the decode kernel: identical caches whenever the two routes produced the
    same code bits, and any bit they disagree on must be one the oracle marks as fragile."""
    w = PARITY_CASES["llama3_8b_gqa"].scaled(batch=2, prompt_len=700, budget=160, decode_steps=0)
    a, b = Case(w), Case(w)
    a.prefill()
    N, G = w.prompt_len, w.group_size
    kc, qc = (codes_np(x).copy() for x in a.gpu.prompt_codes(N))
    b.gpu.reset()
    qcodes = torch.empty((w.n_seq, w.n_kv_heads * G, b.gpu.Wd), dtype=torch.int32, device="cuda")
    rows = [(b.dQ[:, :, t].contiguous(), b.dK[:, :, t].contiguous(), b.dV[:, :, t].contiguous()) for t in range(N)]
    same = True
    for t, (q, k, v) in enumerate(rows):
        vic = b.gpu.decode_step(q, k, v, qcodes_out=qcodes)
        torch.cuda.synchronize()
        step_q = codes_np(qcodes).reshape(w.n_seq, w.n_kv_heads, G, -1)
        step_k = np.take_along_axis(codes_np(b.gpu.codes), vic.cpu().numpy()[:, :, None, None].astype(np.int64), axis=2)[:, :, 0, :]
        for got, want, x in ((step_k, kc[:, :, t], a.K[:, :, t]),) + (((step_q, qc[:, :, t], a.Q[:, :, t].reshape(w.n_seq, w.n_kv_heads, G, -1)),) if t >= w.budget else ()):
            if not np.array_equal(got, want):
                same = False
                _, fragile = oracle.hash_rows(np.ascontiguousarray(x.reshape(-1, w.head_dim)), a.W, w.dtype, want_fragile=True)
                assert not ((got ^ want).reshape(fragile.shape) & ~fragile).any(), f"token {t}: the routes disagree on a bit that is not fragile"
    if same:
        for n in STATE:
            assert torch.equal(getattr(a.gpu, n), getattr(b.gpu, n)), n


DEBUG_SCRIPT = r"""
import sys
sys.path.insert(0, %r); sys.path.insert(0, %r)
from cases import PARITY_CASES
from paper_2412_16187_b200 import device_error_count, binding, workloads as wl
from parity import Case
assert binding.lib()._name.endswith("libhashevict_debug.so")
for name, early in (("tiny", False), ("throughput_batch", False), ("throughput_batch", True), ("protected_gqa", True),
                    ("long_prefill", False), ("llama3_8b_gqa", False)):
    w = PARITY_CASES[name]
    case = Case(w, early_inputs=early)
    case.prefill()
    case.compare_state()
    case.decode(6)
    case.gpu.attend(case.dQ[:, :, 0].contiguous())
    case.gpu.prefill_oneshot(case.dQ, case.dK, case.dV, case.dplen)
    case.gpu.prefill_oneshot_l2(case.dK, case.dV, case.dplen)
    case.gpu.decode_step_l2(case.dK[:, :, 0].contiguous(), case.dV[:, :, 0].contiguous())
w = wl.CONFIGS["long_prefill"].scaled(layers=1, n_kv_heads=2, prompt_len=10240, budget=9830, decode_steps=4)
case = Case(w); case.prefill(); case.compare_state(); case.decode(4)
n = device_error_count()
print("DEVICE_ERRORS", n)
assert n == 0
""" % (ROOT, os.path.join(ROOT, "tests"))


def test_bounds_checking_build_finds_no_index_out_of_range():
    """The library built with -DHE_BOUNDS_CHECK range-checks every slot and token index before using it as an address
    (a failed check skips the access and is counted). Parity cases of every replay and decode kernel run against it in
    a fresh process; the count must stay 0."""
    from paper_2412_16187_b200 import build
    build.build_cuda(debug=True)
    env = dict(os.environ, HE_DEBUG_LIB="1")
    r = subprocess.run([sys.executable, "-c", DEBUG_SCRIPT], env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "DEVICE_ERRORS 0" in r.stdout
