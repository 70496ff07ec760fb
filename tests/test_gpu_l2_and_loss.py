"""he_prefill_oneshot_l2 (the L2-norm comparison policy as a one-shot ranking) and he_attention_loss (Section 4.6)
against the oracle.

L2: the squared norms are fp32 with a fixed summation order on both sides, so they and everything that follows from
them (kept positions, slot contents, scores = -norm2) must match bit for bit; the stored codes are checked through
the usual hash stage. Attention loss: the device sums the dropped attention mass in fp32 with an online maximum, the
oracle in fp64; products of bf16 inputs are exact, so each weight is right to a few 1e-6 relative and the loss, a
ratio of sums of weights, to 2e-5 of its own size plus 1e-6 absolute.
"""
import numpy as np
import pytest
import torch

from paper_2412_16187_b200 import workloads as wl

from cases import PARITY_CASES
from parity import Case, check_hash_stage, codes_np, to_dev

pytestmark = pytest.mark.gpu


def run_l2(w, plen=None):
    case = Case(w)
    if plen is not None:
        case.plen = np.asarray(plen, dtype=np.int32)
        case.dplen = torch.from_numpy(case.plen).cuda()
    Nmax = w.max_prompt_len
    norms = torch.full((w.n_seq, w.n_kv_heads, Nmax), -1.0, dtype=torch.float32, device="cuda")
    case.gpu.prefill_oneshot_l2(case.dK, case.dV, case.dplen, norms_out=norms)
    torch.cuda.synchronize()
    kc, _ = case.gpu.prompt_codes(Nmax)
    kc = codes_np(kc).copy()
    flips = fragile = 0
    for s in range(w.n_seq):
        N = int(case.plen[s])
        f, g = check_hash_stage(case.K[s, :, :N], case.W, w.dtype, kc[s, :, :N])
        flips, fragile = flips + f, fragile + g
        kc[s, :, N:] = 0
    assert flips <= fragile
    want = case.orc.oneshot_l2(kc, case.K, case.V, case.plen, want_norms=True)
    got = norms.cpu().numpy()
    for s in range(w.n_seq):
        N = int(case.plen[s])
        assert np.array_equal(got[s, :, :N], want[s, :, :N]), f"norms differ in sequence {s}"
        assert np.all(got[s, :, N:] == -1.0)
    case.compare_state()
    return case


@pytest.mark.parametrize("name", ["tiny", "llama2_7b_layer", "llama3_8b_gqa", "throughput_batch", "protected_gqa"])
def test_l2_ranking_matches_oracle(name):
    case = run_l2(PARITY_CASES[name])
    w = case.w
    fill = case.gpu.fill.cpu().numpy()
    for s in range(w.n_seq):
        assert np.all(fill[s] == min(int(case.plen[s]), int(w.budgets()[s])))


def test_l2_ranking_short_prompts_and_continues_with_algorithm_1():
    w = PARITY_CASES["throughput_batch"].scaled(batch=4, decode_steps=3)
    b = w.budgets()
    case = run_l2(w, plen=[0, 5, int(b[2]), int(b[3]) + 1])
    case.decode(3)  # the codes it stored make the cache a valid state for he_decode_step


def check_loss(case, q_np, k_full_np):
    w = case.w
    want = case.orc.attention_loss(q_np, k_full_np)
    got = case.gpu.attention_loss(to_dev(q_np, w), to_dev(k_full_np, w))
    torch.cuda.synchronize()
    got = got.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all() and np.all(got >= 0) and np.all(got <= 1 + 1e-6)
    np.testing.assert_allclose(got, want, rtol=2e-5, atol=1e-6)
    return got


@pytest.mark.parametrize("name", ["tiny", "llama2_7b_layer", "llama3_8b_gqa", "throughput_batch"])
@pytest.mark.parametrize("path", ["default", "generic"])
def test_attention_loss_after_each_policy(name, path, monkeypatch):
    w = PARITY_CASES[name]
    if path == "generic":
        if w.dtype != "bf16" or w.head_dim != 128:
            pytest.skip("the default path is already the generic kernel")
        monkeypatch.setenv("HE_DISABLE_ATTEND_MMA", "1")
    q = np.ascontiguousarray(wl.gen_decode_inputs(w, "q", 0, 1)[0])
    case = Case(w)
    case.prefill()  # Algorithm 1
    loss_he = check_loss(case, q, case.K)
    case = run_l2(w)  # comparison policy
    loss_l2 = check_loss(case, q, case.K)
    assert loss_he.shape == loss_l2.shape == (w.n_seq, w.n_kv_heads * w.group_size)
    # queries equal to a stored key: its own weight dominates, the loss becomes small but stays accurate
    k5 = np.ascontiguousarray(case.orc.k_cache[:, :, 5].repeat(w.group_size, axis=1))
    check_loss(case, k5, case.K)


def test_attention_loss_is_zero_when_nothing_was_dropped_and_on_empty_caches():
    w = PARITY_CASES["llama3_8b_gqa"]
    case = Case(w)
    q = np.ascontiguousarray(wl.gen_decode_inputs(w, "q", 0, 1)[0])
    out = case.gpu.attention_loss(to_dev(q, w), case.dK)
    torch.cuda.synchronize()
    assert not out.cpu().numpy().any()  # nothing seen yet
    short = np.minimum(case.plen, w.budgets() - 1).astype(np.int32)
    case.plen = short
    case.dplen = torch.from_numpy(short).cuda()
    case.prefill()
    out = case.gpu.attention_loss(to_dev(q, w), case.dK)
    torch.cuda.synchronize()
    assert not out.cpu().numpy().any()  # every token is still cached


@pytest.mark.parametrize("name", ["tiny", "llama3_8b_gqa", "throughput_batch", "protected_gqa"])
def test_l2_decode_steps_match_oracle(name):
    w = PARITY_CASES[name]
    case = run_l2(w)
    steps = 12
    dk, dv = wl.gen_decode_inputs(w, "k", 0, steps), wl.gen_decode_inputs(w, "v", 0, steps)
    dk[5] = dk[2]  # a repeated key: equal norms, the lower slot must leave first when both are candidates
    gk, gv = to_dev(dk, w), to_dev(dv, w)
    victim = torch.empty((w.n_seq, w.n_kv_heads), dtype=torch.int32, device="cuda")
    evicted = torch.empty_like(victim)
    for i in range(steps):
        case.gpu.decode_step_l2(gk[i], gv[i], victim, evicted)
        torch.cuda.synchronize()
        ovic, oev = case.orc.step_l2(np.ascontiguousarray(dk[i]), np.ascontiguousarray(dv[i]))
        assert np.array_equal(victim.cpu().numpy(), ovic), f"victims differ at step {i}"
        assert np.array_equal(evicted.cpu().numpy(), oev), f"evicted positions differ at step {i}"
    case.compare_state()


def test_l2_decode_from_an_empty_cache_appends_then_evicts():
    w = PARITY_CASES["tiny"]
    case = Case(w)
    steps = int(w.budgets().max()) + 9
    dk, dv = wl.gen_decode_inputs(w, "k", 0, steps), wl.gen_decode_inputs(w, "v", 0, steps)
    gk, gv = to_dev(dk, w), to_dev(dv, w)
    for i in range(steps):
        vic = case.gpu.decode_step_l2(gk[i], gv[i])
        ovic, _ = case.orc.step_l2(np.ascontiguousarray(dk[i]), np.ascontiguousarray(dv[i]))
        assert np.array_equal(vic.cpu().numpy(), ovic)
    case.compare_state()
