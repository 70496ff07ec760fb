"""he_prefill_compress_noalloc against he_prefill_compress (collected last on purpose: a failure here must not
hide the other tests from a run that stops at the first failure).

The variant exists for callers that cannot allocate device memory for the prompt-code workspace; it must give
exactly what the ordinary entry point gives. Two calls in a row are checked, the second on different prompts, so
that whatever the first call left in the shared built-in scratch is shown not to matter."""
import numpy as np
import pytest
import torch

from cases import PARITY_CASES
from paper_2412_16187_b200 import HashEvictError
from parity import Case

pytestmark = pytest.mark.gpu

STATE = ("codes", "pos", "fill", "next_pos", "scores", "k_cache", "v_cache")


def test_noalloc_prefill_matches_ordinary_prefill_twice_in_a_row():
    w = PARITY_CASES["llama3_8b_gqa"].scaled(batch=2, prompt_len=900, budget=333, decode_steps=0)
    ref, new = Case(w), Case(w)
    # first call: full prompts
    ref.gpu.prefill_compress(ref.dQ, ref.dK, ref.dV, ref.dplen)
    new.gpu.prefill_compress_noalloc(new.dQ, new.dK, new.dV, new.dplen)
    torch.cuda.synchronize()
    for name in STATE:
        assert torch.equal(getattr(ref.gpu, name), getattr(new.gpu, name)), f"first call: {name}"
    assert int(ref.gpu.fill.min()) == 333
    # the call itself takes no device memory: neither from the driver nor from torch's pool
    torch.cuda.synchronize()
    free_before, alloc_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    new.gpu.prefill_compress_noalloc(new.dQ, new.dK, new.dV, new.dplen)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == alloc_before
    # second call right after it: shorter, ragged prompts (one below its budget), reversed token order as new data
    plen = torch.tensor([517, 120], dtype=torch.int32, device="cuda")
    q2, k2, v2 = (t.flip(2).contiguous() for t in (ref.dQ, ref.dK, ref.dV))
    ref.gpu.prefill_compress(q2, k2, v2, plen)
    new.gpu.prefill_compress_noalloc(q2, k2, v2, plen)
    torch.cuda.synchronize()
    for name in STATE:
        assert torch.equal(getattr(ref.gpu, name), getattr(new.gpu, name)), f"second call: {name}"
    assert ref.gpu.fill.cpu()[:, 0].tolist() == [333, 120]


def test_noalloc_prefill_rejects_prompts_beyond_the_builtin_scratch():
    w = PARITY_CASES["throughput_batch"].scaled(batch=2)
    case = Case(w)
    too_long = 16 * 2 ** 20 // (w.n_units * (1 + w.group_size) * 2 * 4) + 64  # prompt codes would exceed 16 MiB
    with pytest.raises(HashEvictError, match="built-in scratch"):
        case.gpu.prefill_compress_noalloc(case.dQ, case.dK, case.dV, case.dplen, max_prompt_len=too_long)
