"""he_attend (Eq. 1 over the compressed cache, Algorithm 1 line 6) against the fp64 oracle.

The cache is brought to the same state on both sides first (prefill + a few decode steps, compared bit for bit by
the parity helpers), so any difference here comes from the attention arithmetic alone. Tolerance: the device carries
scores, softmax and sums in fp32 (bf16 products are exact), which leaves each softmax weight with a relative error
of a few 1e-6; outputs are weighted means of V rows, so they must agree to 2e-5 * max|V| of the unit.
"""
import numpy as np
import pytest
import torch

from paper_2412_16187_b200 import HashEvictError
from paper_2412_16187_b200 import workloads as wl

from cases import PARITY_CASES
from parity import Case, to_dev

pytestmark = pytest.mark.gpu

TOL = 2e-5


def check_attend(case, q_np):
    w = case.w
    want = case.orc.attend(q_np)
    got = case.gpu.attend(to_dev(q_np, w))
    torch.cuda.synchronize()
    got = got.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    V = wl.as_f64(w, case.orc.v_cache)
    worst = 0.0
    for s in range(w.n_seq):
        for h in range(w.n_kv_heads):
            f = int(case.orc.fill[s, h])
            rows = slice(h * w.group_size, (h + 1) * w.group_size)
            if f == 0:
                assert not got[s, rows].any()
                continue
            vmax = np.abs(V[s, h, :f]).max()
            err = np.abs(got[s, rows] - want[s, rows]).max() / vmax
            worst = max(worst, err)
            assert err <= TOL, f"unit ({s},{h}) fill {f}: error {err:.3g} of max|V|"
    return worst


@pytest.mark.parametrize("name", list(PARITY_CASES))
@pytest.mark.parametrize("path", ["default", "generic"])
def test_attend_after_prefill_and_decode(name, path, monkeypatch):
    w = PARITY_CASES[name]
    if path == "generic":
        if w.dtype != "bf16" or w.head_dim != 128:
            pytest.skip("the default path is already the generic kernel")
        monkeypatch.setenv("HE_DISABLE_ATTEND_MMA", "1")
    case = Case(w)
    case.prefill()
    case.decode(3)
    q = wl.gen_decode_inputs(w, "q", 7, 8)[0]
    check_attend(case, np.ascontiguousarray(q))
    # queries aligned with stored keys give peaked weights: the running maximum moves a lot
    k5 = case.orc.k_cache[:, :, 5].repeat(w.group_size, axis=1)
    check_attend(case, np.ascontiguousarray(k5))


def test_attend_on_empty_and_partly_filled_units():
    w = PARITY_CASES["llama3_8b_gqa"]
    case = Case(w)
    q = np.ascontiguousarray(wl.gen_decode_inputs(w, "q", 3, 4)[0])
    out = case.gpu.attend(to_dev(q, w))
    torch.cuda.synchronize()
    assert not out.cpu().numpy().any()  # nothing stored yet
    # prompts of 0, 1 and 37 tokens: an empty unit, a single slot (the output is that V row) and a ragged group
    plen = np.array([0, 1, 37], dtype=np.int32)[: w.n_seq]
    case.plen = plen
    case.dplen = torch.from_numpy(plen).cuda()
    case.prefill()
    check_attend(case, q)
    got = case.gpu.attend(to_dev(q, w)).cpu().numpy()
    V = wl.as_f64(w, case.orc.v_cache)
    for h in range(w.n_kv_heads):
        for g in range(w.group_size):
            np.testing.assert_allclose(got[1, h * w.group_size + g], V[1, h, 0], rtol=1e-6, atol=1e-7)


def test_attend_rejects_bad_arguments():
    w = PARITY_CASES["tiny"]
    case = Case(w)
    q = to_dev(np.ascontiguousarray(wl.gen_decode_inputs(w, "q", 3, 4)[0]), w)
    with pytest.raises(HashEvictError, match="aligned"):
        case.gpu.attend(q.reshape(-1)[1:])  # not 16-byte aligned
