"""he_prefill_oneshot (the averaged-Hamming ranking of Appendix C as a prompt-compression variant) against the oracle.

Same staging as the other parity tests: the device's Eq. 2 codes are checked against the oracle's under the
fragile-bit rule, then the oracle ranks on the DEVICE's codes, so the summed distances, the kept positions, the
stored codes, scores, K / V rows, fill and next_pos must match bit for bit (the score is one fp32 division of two
exactly representable integers on both sides).
"""
import numpy as np
import pytest
import torch

from paper_2412_16187_b200 import HashEvictError
from paper_2412_16187_b200 import workloads as wl

from cases import PARITY_CASES
from parity import Case, check_hash_stage, codes_np

pytestmark = pytest.mark.gpu


def run_oneshot(w, plen=None):
    case = Case(w)
    if plen is not None:
        case.plen = np.asarray(plen, dtype=np.int32)
        case.dplen = torch.from_numpy(case.plen).cuda()
    Nmax = w.max_prompt_len
    sums = torch.full((w.n_seq, w.n_kv_heads, Nmax), -1, dtype=torch.int64, device="cuda")
    case.gpu.prefill_oneshot(case.dQ, case.dK, case.dV, case.dplen, sums_out=sums)
    torch.cuda.synchronize()
    kc, qc = case.gpu.prompt_codes(Nmax)
    kc, qc = codes_np(kc).copy(), codes_np(qc).copy()
    flips = fragile = 0
    for s in range(w.n_seq):
        N = int(case.plen[s])
        f, g = check_hash_stage(case.K[s, :, :N], case.W, w.dtype, kc[s, :, :N])
        flips, fragile = flips + f, fragile + g
        qs = case.Q[s, :, :N].reshape(w.n_kv_heads, w.group_size, N, w.head_dim).transpose(0, 2, 1, 3)
        f, g = check_hash_stage(qs, case.W, w.dtype, qc[s, :, :N])  # every prompt query is hashed for this variant
        flips, fragile = flips + f, fragile + g
        kc[s, :, N:] = 0
        qc[s, :, N:] = 0
    assert flips <= fragile
    want = case.orc.oneshot_codes(kc, qc, case.K, case.V, case.plen, want_sums=True)
    got = sums.cpu().numpy()
    for s in range(w.n_seq):
        N = int(case.plen[s])
        assert np.array_equal(got[s, :, :N], want[s, :, :N]), f"summed distances differ in sequence {s}"
        assert np.all(got[s, :, N:] == -1)  # entries beyond the prompt are not written
    case.compare_state()
    return case


@pytest.mark.parametrize("name", ["tiny", "llama2_7b_layer", "llama3_8b_gqa", "throughput_batch", "protected_gqa", "protected_tiny"])
def test_oneshot_matches_oracle(name):
    w = PARITY_CASES[name]
    if w.max_prompt_len > 2048:  # the oracle's double sum is quadratic in the prompt length
        w = w.scaled(prompt_len=2048)
    case = run_oneshot(w)
    fill = case.gpu.fill.cpu().numpy()
    budgets, plen = w.budgets(), case.plen
    for s in range(w.n_seq):
        assert np.all(fill[s] == min(int(plen[s]), int(budgets[s])))


def test_oneshot_short_empty_and_odd_shapes():
    w = PARITY_CASES["throughput_batch"].scaled(batch=4)
    b = w.budgets()
    run_oneshot(w, plen=[0, 5, int(b[2]), int(b[3]) + 1])
    w = wl.CONFIGS["throughput_batch"].scaled(batch=2, budget_lo=130, budget_hi=300, group_size=3, hash_bits=40)
    run_oneshot(w)
    w = wl.CONFIGS["llama3_8b_gqa"].scaled(batch=1, prompt_len=777, budget=129, hash_bits=4)
    run_oneshot(w)  # four-bit codes: many equal averages, the index decides


def test_oneshot_differs_from_algorithm_1_and_decode_continues():
    w = PARITY_CASES["llama3_8b_gqa"].scaled(prompt_len=1024, decode_steps=4)
    case = run_oneshot(w)
    one = case.gpu.pos.cpu().numpy().copy()
    case.decode(4)  # the cache it leaves is a valid starting state for Algorithm 1
    seq = Case(w)
    seq.prefill()
    assert not np.array_equal(one, seq.gpu.pos.cpu().numpy())  # a different policy keeps different tokens


def test_oneshot_rejects_small_workspace_and_long_prompts():
    w = PARITY_CASES["tiny"]
    case = Case(w)
    case.gpu._ws = None
    with pytest.raises(HashEvictError, match="32768"):
        case.gpu.prefill_oneshot(case.dQ, case.dK, case.dV, case.dplen, max_prompt_len=40000)
