"""The byte-packed code table (HE_FLAG_PACKED_CODES: ceil(b/8) bytes per slot, 1 byte at b <= 8 as Section 4.7 counts
it) against the oracle, and against the word layout of the same library.

The oracle knows one layout (32-bit words); the binding widens the packed table to words for the comparison, so the
staging of the other parity tests applies unchanged: device codes under the fragile-bit rule, then every integer
result bit for bit.
"""
import numpy as np
import pytest
import torch

from paper_2412_16187_b200 import HashEvictCache, HashEvictError
from paper_2412_16187_b200 import workloads as wl

from cases import PARITY_CASES
from parity import Case

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("b", [4, 8, 13, 16, 24, 32])
@pytest.mark.parametrize("base", ["llama3_8b_gqa", "llama2_7b_layer", "protected_gqa"])
def test_packed_prefill_then_decode_matches_oracle(base, b):
    w = PARITY_CASES[base].scaled(batch=2, prompt_len=700, budget=261, decode_steps=10, hash_bits=b)
    case = Case(w, packed_codes=True)
    assert case.gpu.codes_storage.dtype == torch.uint8 and case.gpu.codes_storage.shape[-1] == (b + 7) // 8
    assert case.gpu.Cmax % 16 == 0
    case.prefill()
    case.compare_state()
    case.decode(10, check_every=5)


def test_packed_generic_group_ragged_budgets_and_scores_off():
    w = PARITY_CASES["protected_gqa"].scaled(group_size=3, hash_bits=11, batch=3, prompt_len=300, budget=97, decode_steps=16)
    case = Case(w, packed_codes=True)
    case.prefill()
    case.compare_state()
    case.decode(16)
    w2 = wl.CONFIGS["throughput_batch"].scaled(batch=6, budget_lo=40, budget_hi=130, prompt_factor=2, decode_steps=6, hash_bits=8)
    case2 = Case(w2, write_scores=False, packed_codes=True)
    case2.prefill()
    q, k, v = (torch.from_numpy(wl.gen_decode_inputs(w2, n, 0, 6).view(np.int16)).cuda().view(torch.bfloat16) for n in ("q", "k", "v"))
    for i in range(6):
        case2.gpu.decode_step(q[i], k[i], v[i])
    case2.compare_state(("fill",))
    assert not case2.gpu.scores.any()  # the flag is off: neither prefill nor decode wrote a score


def test_packed_decode_from_an_empty_cache():
    """Appends first, evictions once the budget is reached: the decode kernel alone builds the table byte by byte."""
    w = PARITY_CASES["tiny"].scaled(hash_bits=8, decode_steps=80)
    case = Case(w, packed_codes=True)
    case.gpu.reset()
    case.compare_state(("codes", "pos", "fill", "next_pos"))
    case.decode(int(w.budgets().max()) + 12, check_every=8)


@pytest.mark.parametrize("b", [8, 16, 24])
def test_packed_and_word_layouts_agree_at_a_tensor_core_shape(b):
    """Budget large enough for the tensor-core replay: both layouts must leave the same state, then decode alike."""
    w = wl.CONFIGS["throughput_batch"].scaled(batch=2, budget_lo=1300, budget_hi=2100, prompt_factor=2, decode_steps=8, hash_bits=b)
    W = torch.from_numpy(wl.gen_W(w))
    K, Q, V = (torch.from_numpy(wl.gen_tokens(w, n, 0, w.n_seq, 0, w.max_prompt_len).view(np.int16)).cuda().view(torch.bfloat16)
               for n in ("k", "q", "v"))
    plen = torch.from_numpy(w.prompt_lens()).cuda()
    dq, dk, dv = (torch.from_numpy(wl.gen_decode_inputs(w, n, 0, 8).view(np.int16)).cuda().view(torch.bfloat16) for n in ("q", "k", "v"))
    states = []
    for packed in (False, True):
        c = HashEvictCache(w.n_seq, w.n_kv_heads, w.group_size, w.head_dim, b, w.budgets(), W, n_sink=w.n_sink,
                           n_recent=w.n_recent, packed_codes=packed, max_budget=2112)
        c.prefill_compress(Q, K, V, plen)
        vics = []
        for i in range(8):
            vics.append(c.decode_step(dq[i], dk[i], dv[i]).clone())
        torch.cuda.synchronize()
        states.append([c.codes.clone(), c.pos.clone(), c.scores.clone(), c.fill.clone(), c.k_cache.clone()] + vics)
    for x, y in zip(*states):
        assert torch.equal(x, y)
    assert int(states[0][3].min()) >= 1300  # the caches are full: every decode step evicted


def test_packed_oneshot_variants_store_packed_codes():
    w = PARITY_CASES["llama3_8b_gqa"].scaled(batch=2, prompt_len=500, budget=128, hash_bits=16)
    a, b_ = Case(w), Case(w, packed_codes=True)
    for c in (a, b_):
        c.gpu.prefill_oneshot(c.dQ, c.dK, c.dV, c.dplen)
    torch.cuda.synchronize()
    assert torch.equal(a.gpu.codes[:, :, :128], b_.gpu.codes[:, :, :128]) and torch.equal(a.gpu.pos[:, :, :128], b_.gpu.pos[:, :, :128])
    assert int(b_.gpu.codes.abs().sum()) > 0


def test_packed_layout_rejects_what_it_cannot_hold():
    w = PARITY_CASES["tiny"]
    W = torch.from_numpy(wl.gen_W(w.scaled(hash_bits=40)))
    with pytest.raises(HashEvictError, match="packed codes"):
        HashEvictCache(1, 1, 1, w.head_dim, 40, [32], W, packed_codes=True).reset()
