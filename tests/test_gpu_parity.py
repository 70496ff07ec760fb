"""GPU-vs-oracle parity through the C ABI (run with -m gpu on a B200). Integer results bit-exact;
scores are integers stored as fp32, so the 1e-6 relative bound is met with equality."""
import numpy as np
import pytest
import torch

import oracle
from cases import PARITY_CASES
from paper_2412_16187_b200 import HashEvictCache, HashEvictError, hash_keys
from paper_2412_16187_b200 import workloads as wl
from parity import Case, check_hash_stage, codes_np, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,d,b,rows", [
    ("f32", 64, 8, 1000), ("bf16", 128, 32, 4097), ("bf16", 128, 64, 2500), ("bf16", 128, 16, 129), ("f32", 40, 24, 77),
    ("bf16", 256, 40, 300), ("f32", 8, 1, 5), ("bf16", 128, 64, 1), ("bf16", 128, 33, 128),
])
def test_hash_keys_stage_h(dtype, d, b, rows):
    w = wl.Workload("h", 17, 1, 1, 1, 1, d, dtype, b, rows, 4, 0, wl.KIND_DRIFT if d >= 64 else wl.KIND_IID)
    W = wl.gen_W(w)
    x = wl.gen_tokens(w, "k", 0, 1, 0, rows)[0, 0]
    got = codes_np(hash_keys(to_dev(x, w), torch.from_numpy(W).cuda()))
    flips, fragile = check_hash_stage(x, W, dtype, got)
    assert flips <= fragile
    if b % 32:
        assert np.all(got[:, -1] >> np.uint32(b % 32) == 0)


def test_hash_keys_strided_rows_and_empty():
    w = wl.Workload("h", 3, 1, 1, 1, 1, 128, "bf16", 32, 64, 4, 0, wl.KIND_IID)
    W = wl.gen_W(w)
    x = wl.gen_tokens(w, "k", 0, 1, 0, 64)[0, 0]
    wide = torch.zeros((64, 256), dtype=torch.bfloat16, device="cuda")
    wide[:, :128] = to_dev(x, w)
    got = codes_np(hash_keys(wide[:, :128], torch.from_numpy(W).cuda()))
    check_hash_stage(x, W, "bf16", got)
    assert hash_keys(wide[:0, :128], torch.from_numpy(W).cuda()).shape == (0, 1)


def test_hash_sign_of_zero_is_one():
    W = torch.randn(64, 48, device="cuda")
    x = torch.zeros(3, 64, device="cuda")
    x[1] = -0.0
    got = codes_np(hash_keys(x, W))
    assert got.tolist() == [[0xFFFFFFFF, 0xFFFF]] * 3


@pytest.mark.parametrize("name", list(PARITY_CASES))
def test_prefill_then_decode_matches_oracle(name):
    w = PARITY_CASES[name]
    case = Case(w)
    flips, fragile = case.prefill()
    case.compare_state()
    f2, g2 = case.decode(w.decode_steps, check_every=8)
    assert flips + f2 <= fragile + g2
    if name == "tiny":  # 6144 + hashed decode bits, ~0.4 fragile expected: end to end with no exception at seed 0
        assert flips + f2 == 0


def test_decode_from_empty_cache_equals_prefill():
    """he_reset + N decode steps == he_prefill_compress (Section 3: both are Algorithm 1 in token order)."""
    w = PARITY_CASES["tiny"].scaled(n_sink=1, n_recent=2)
    a, b = Case(w), Case(w)
    a.prefill()
    b.gpu.reset()
    b.orc.reset()
    N = w.prompt_len
    for t in range(N):
        b.gpu.decode_step(b.dQ[:, :, t].contiguous(), b.dK[:, :, t].contiguous(), b.dV[:, :, t].contiguous())
    torch.cuda.synchronize()
    for name in ("codes", "pos", "fill", "next_pos", "scores", "k_cache", "v_cache"):
        assert torch.equal(getattr(a.gpu, name), getattr(b.gpu, name)), name


def test_short_and_empty_prompts():
    w = PARITY_CASES["throughput_batch"].scaled(batch=4, decode_steps=3)
    case = Case(w)
    case.plen = np.array([0, 5, int(w.budgets()[2]), int(w.budgets()[3]) + 1], dtype=np.int32)
    case.dplen = torch.from_numpy(case.plen).cuda()
    case.prefill()
    case.compare_state()
    assert case.gpu.fill.cpu().numpy()[:, 0].tolist() == [0, 5, int(w.budgets()[2]), int(w.budgets()[3])]
    # decode inputs continue each sequence's own token axis; here only the mechanics matter
    case.decode(3)


def test_scores_flag_off_leaves_scores_untouched():
    w = PARITY_CASES["tiny"]
    case = Case(w, write_scores=False)
    case.prefill()
    case.compare_state(("codes", "pos", "fill", "next_pos", "k_cache", "v_cache"))
    assert not case.gpu.scores.any()


def test_generic_group_size_and_odd_bits():
    w = PARITY_CASES["protected_gqa"].scaled(group_size=3, hash_bits=40, batch=2, prompt_len=300, budget=97, decode_steps=16)
    case = Case(w)
    case.prefill()
    case.compare_state()
    case.decode(16)


def test_large_budget_uses_wider_blocks():
    w = wl.CONFIGS["long_prefill"].scaled(layers=1, n_kv_heads=2, prompt_len=10240, budget=9830, decode_steps=6)
    case = Case(w)
    case.prefill()
    case.compare_state()
    case.decode(6)


def test_bad_arguments_are_rejected():
    W = torch.randn(128, 32, device="cuda")
    with pytest.raises(HashEvictError, match="hash_bits"):
        hash_keys(torch.zeros(4, 128, device="cuda"), torch.randn(128, 65, device="cuda"))
    with pytest.raises(HashEvictError, match="head_dim"):
        hash_keys(torch.zeros(4, 12, device="cuda"), torch.randn(12, 8, device="cuda"))
    c = HashEvictCache(1, 1, 1, 128, 32, [8], W)
    with pytest.raises(HashEvictError, match="null"):
        c.decode_step(None, torch.zeros(1, 1, 128, device="cuda"), torch.zeros(1, 1, 128, device="cuda"))
    with pytest.raises(HashEvictError, match="group_size"):
        HashEvictCache(1, 1, 9, 128, 32, [8], W).reset()


def test_host_buffer_variants_match_device_calls():
    w = PARITY_CASES["protected_tiny"]
    a, b = Case(w), Case(w)
    a.prefill()
    from paper_2412_16187_b200 import decode_staging_bytes, prefill_staging_bytes
    Nmax = w.max_prompt_len
    staging = torch.empty(prefill_staging_bytes(b.gpu.cfg, Nmax), dtype=torch.uint8, device="cuda")
    fill_host = torch.empty((w.n_seq, w.n_kv_heads), dtype=torch.int32).pin_memory()
    hq, hk, hv = (torch.from_numpy(x).pin_memory() for x in (b.Q, b.K, b.V))
    b.gpu.prefill_compress_host(hq, hk, hv, torch.from_numpy(b.plen), Nmax, fill_host, staging)
    assert torch.equal(fill_host, a.gpu.fill.cpu())
    for name in ("codes", "pos", "scores", "k_cache", "v_cache"):
        assert torch.equal(getattr(a.gpu, name), getattr(b.gpu, name)), name
    dq, dk, dv = (wl.gen_decode_inputs(w, x, 0, 1)[0] for x in "qkv")
    va = a.gpu.decode_step(to_dev(dq, w), to_dev(dk, w), to_dev(dv, w))
    st = torch.empty(decode_staging_bytes(b.gpu.cfg), dtype=torch.uint8, device="cuda")
    vb = torch.empty((w.n_seq, w.n_kv_heads), dtype=torch.int32).pin_memory()
    b.gpu.decode_step_host(torch.from_numpy(dq).pin_memory(), torch.from_numpy(dk).pin_memory(),
                           torch.from_numpy(dv).pin_memory(), vb, st)
    assert torch.equal(va.cpu(), vb)
    assert torch.equal(a.gpu.codes, b.gpu.codes) and torch.equal(a.gpu.k_cache, b.gpu.k_cache)


def test_enqueued_host_steps_on_two_streams_match_device_calls():
    """he_decode_step_host_enqueue: two caches on two streams, several steps in flight, one synchronise at the end."""
    from paper_2412_16187_b200 import decode_staging_bytes
    w = PARITY_CASES["protected_tiny"]
    steps = 12
    ref, x, y = Case(w), Case(w), Case(w)
    for c in (ref, x, y):
        c.gpu.prefill_compress(c.dQ, c.dK, c.dV, c.dplen)
    dq, dk, dv = (wl.gen_decode_inputs(w, n, 0, steps) for n in "qkv")
    want = [ref.gpu.decode_step(to_dev(dq[i], w), to_dev(dk[i], w), to_dev(dv[i], w)).cpu() for i in range(steps)]
    hq, hk, hv = (torch.from_numpy(t).pin_memory() for t in (dq, dk, dv))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    stagings = [torch.empty(decode_staging_bytes(x.gpu.cfg), dtype=torch.uint8, device="cuda") for _ in range(2)]
    got = torch.empty((2, steps, w.n_seq, w.n_kv_heads), dtype=torch.int32).pin_memory()
    torch.cuda.synchronize()
    for i in range(steps):
        for ci, c in enumerate((x, y)):
            c.gpu.decode_step_host_enqueue(hq[i], hk[i], hv[i], got[ci, i], stagings[ci], stream=streams[ci])
    torch.cuda.synchronize()
    for ci, c in enumerate((x, y)):
        for i in range(steps):
            assert torch.equal(got[ci, i], want[i]), (ci, i)
        for name in ("codes", "pos", "scores", "k_cache", "v_cache", "fill", "next_pos"):
            assert torch.equal(getattr(ref.gpu, name), getattr(c.gpu, name)), name


def test_host_block_steps_match_device_calls():
    """he_decode_step_host_block_enqueue: a step's q, k, v in one pinned block at the documented offsets, one copy in."""
    from paper_2412_16187_b200 import decode_staging_bytes
    w = PARITY_CASES["protected_tiny"]
    steps = 6
    ref, x = Case(w), Case(w)
    for c in (ref, x):
        c.gpu.prefill_compress(c.dQ, c.dK, c.dV, c.dplen)
    dq, dk, dv = (wl.gen_decode_inputs(w, n, 0, steps) for n in "qkv")
    want = [ref.gpu.decode_step(to_dev(dq[i], w), to_dev(dk[i], w), to_dev(dv[i], w)).cpu() for i in range(steps)]
    nbytes, offs = x.gpu.host_block_layout()
    assert offs[0] == 0 and offs[1] % 256 == 0 and offs[2] % 256 == 0 and nbytes == offs[2] + dk[0].nbytes
    block = torch.zeros((steps, (nbytes + 255) // 256 * 256), dtype=torch.uint8).pin_memory()
    for i in range(steps):
        for o, t in zip(offs, (dq[i], dk[i], dv[i])):
            block[i, o:o + t.nbytes] = torch.from_numpy(np.ascontiguousarray(t).view(np.uint8).reshape(-1))
    st = torch.empty(decode_staging_bytes(x.gpu.cfg), dtype=torch.uint8, device="cuda")
    got = torch.empty((steps, w.n_seq, w.n_kv_heads), dtype=torch.int32).pin_memory()
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    for i in range(steps):
        x.gpu.decode_step_host_block_enqueue_raw(block[i].data_ptr(), got[i].data_ptr(), st.data_ptr(), st.numel(), stream.cuda_stream)
    torch.cuda.synchronize()
    for i in range(steps):
        assert torch.equal(got[i], want[i]), i
    for name in ("codes", "pos", "scores", "k_cache", "v_cache", "fill", "next_pos"):
        assert torch.equal(getattr(ref.gpu, name), getattr(x.gpu, name)), name


def _sampled_full_size_check(w, seqs, decode_steps, early_inputs=False):
    """Full-size workload on the device in the launch configuration the benchmark times; the oracle replays only
    the sampled sequences (all their KV heads) on the device's codes and must reproduce their final state."""
    import oracle as orc
    from parity import raw_np, torch_dtype
    Nmax = w.max_prompt_len
    W = wl.gen_W(w)
    plen, budgets = w.prompt_lens(), w.budgets()
    gpu = HashEvictCache(w.n_seq, w.n_kv_heads, w.group_size, w.head_dim, w.hash_bits, budgets, torch.from_numpy(W),
                         dtype=torch_dtype(w), early_inputs=early_inputs)
    tdt = torch_dtype(w)
    dK = torch.zeros((w.n_seq, w.n_kv_heads, Nmax, w.head_dim), dtype=tdt, device="cuda")
    dV = torch.zeros_like(dK)
    dQ = torch.zeros((w.n_seq, w.n_kv_heads * w.group_size, Nmax, w.head_dim), dtype=tdt, device="cuda")
    for s in range(w.n_seq):
        n = int(plen[s])
        dK[s, :, :n] = to_dev(wl.gen_tokens(w, "k", s, 1, 0, n)[0], w)
        dV[s, :, :n] = to_dev(wl.gen_tokens(w, "v", s, 1, 0, n)[0], w)
        dQ[s, :, :n] = to_dev(wl.gen_tokens(w, "q", s, 1, 0, n)[0], w)
    gpu.prefill_compress(dQ, dK, dV, torch.from_numpy(plen).cuda())
    torch.cuda.synchronize()
    kc_all, qc_all = gpu.prompt_codes(Nmax)
    G, Wd = w.group_size, gpu.Wd
    dq, dk, dv = (wl.gen_decode_inputs(w, x, 0, decode_steps) for x in "qkv")
    gq, gk, gv = to_dev(dq, w), to_dev(dk, w), to_dev(dv, w)
    victim = torch.empty((w.n_seq, w.n_kv_heads), dtype=torch.int32, device="cuda")
    qcodes = torch.empty((w.n_seq, w.n_kv_heads * G, Wd), dtype=torch.int32, device="cuda")
    oracles = {}
    for s in seqs:
        n = int(plen[s])
        oc = orc.OracleCache(1, w.n_kv_heads, G, w.head_dim, w.hash_bits, gpu.Cmax, budgets[s:s + 1], w.dtype, threads=8)
        kc = codes_np(kc_all[s:s + 1, :, :n]).copy()
        qc = codes_np(qc_all[s:s + 1, :, :n]).copy()
        qc[:, :, :min(n, int(budgets[s]))] = 0
        Ks, Vs = raw_np(dK[s:s + 1, :, :n]), raw_np(dV[s:s + 1, :, :n])
        check_hash_stage(Ks[0], W, w.dtype, kc[0])
        oc.prefill_codes(kc, qc, np.ascontiguousarray(Ks), np.ascontiguousarray(Vs), plen[s:s + 1])
        oracles[s] = oc
    for i in range(decode_steps):
        gpu.decode_step(gq[i], gk[i], gv[i], victim_out=victim, qcodes_out=qcodes)
        torch.cuda.synchronize()
        vic = victim.cpu().numpy()
        gcodes = codes_np(gpu.codes)
        for s, oc in oracles.items():
            kc = np.take_along_axis(gcodes[s:s + 1], vic[s:s + 1, :, None, None].astype(np.int64), axis=2)[:, :, 0, :]
            ovic, _ = oc.step_codes(codes_np(qcodes[s:s + 1]), kc, np.ascontiguousarray(dk[i, s:s + 1]),
                                    np.ascontiguousarray(dv[i, s:s + 1]))
            assert np.array_equal(ovic, vic[s:s + 1]), f"victims differ: sequence {s}, decode step {i}"
    for s, oc in oracles.items():
        f = int(oc.fill[0, 0])
        assert np.array_equal(codes_np(gpu.codes[s]), oc.codes[0]) and np.array_equal(gpu.pos[s].cpu().numpy(), oc.pos[0])
        assert np.array_equal(gpu.scores[s].cpu().numpy(), oc.scores[0])
        assert np.array_equal(raw_np(gpu.k_cache[s, :, :f]), oc.k_cache[0, :, :f])
        assert np.array_equal(raw_np(gpu.v_cache[s, :, :f]), oc.v_cache[0, :, :f])


def test_full_size_throughput_batch_sampled_sequences():
    """Configuration 5 in full on the device; the oracle follows 8 of the 64 sequences (shortest, median and longest
    budget plus five seeded picks) through the prefill and 64 decode steps."""
    w = wl.CONFIGS["throughput_batch"]
    b = w.budgets()
    order = np.argsort(b, kind="stable")
    picks = [int(order[0]), int(order[len(order) // 2]), int(order[-1])]
    rng = np.random.default_rng(5)
    for s in rng.permutation(w.n_seq):
        if len(picks) == 8:
            break
        if int(s) not in picks:
            picks.append(int(s))
    _sampled_full_size_check(w, picks, decode_steps=64)


def test_full_size_throughput_batch_sampled_sequences_early_inputs():
    w = wl.CONFIGS["throughput_batch"]
    order = np.argsort(w.budgets(), kind="stable")
    _sampled_full_size_check(w, [int(order[1]), int(order[-2])], decode_steps=24, early_inputs=True)


def test_full_size_long_prefill_sampled_layer():
    # full per-unit size (32768-token prompt, 9830 slots, 22938 evicting steps), 4 of the 32 folded layers on the
    # device, two of them replayed by the oracle, 16 decode steps
    w = wl.CONFIGS["long_prefill"].scaled(layers=4)
    _sampled_full_size_check(w, [1, 2], decode_steps=16)


def test_prefill_with_token_major_strided_inputs():
    """q/k/v stored [B, N, heads, d] (token-major, as a fused QKV projection writes them) and handed over as strided
    views: the tensor-core projection's tensor map and the gather must follow the strides."""
    w = PARITY_CASES["llama3_8b_gqa"].scaled(batch=2, prompt_len=1500, budget=300, decode_steps=0)
    a, b = Case(w), Case(w)
    a.prefill()
    a.compare_state()
    tm = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)  # same values, token-major storage
    q, k, v = tm(b.dQ), tm(b.dK), tm(b.dV)
    assert not k.is_contiguous() and k.stride(2) == w.n_kv_heads * w.head_dim
    b.gpu.prefill_compress(q, k, v, b.dplen)
    torch.cuda.synchronize()
    for name in ("codes", "pos", "fill", "next_pos", "scores", "k_cache", "v_cache"):
        assert torch.equal(getattr(a.gpu, name), getattr(b.gpu, name)), name


def test_no_kernel_gave_up_on_a_bounded_wait():
    from paper_2412_16187_b200 import device_error_count
    x = torch.randn(20000, 128, device="cuda").to(torch.bfloat16)
    hash_keys(x, torch.randn(128, 64, device="cuda"))
    assert device_error_count() == 0


@pytest.mark.parametrize("batch,dtype", [(512, "bf16"), (515, "bf16"), (512, "f32")],
                         ids=["whole_tiles", "ragged_tiles", "fp32_cuda_cores"])
def test_large_batch_decode_hashes_new_rows_in_bulk(batch, dtype):
    """About 4100 units x (G + 1) = 20500 new rows per step: he_decode_step hashes them with the bulk projection kernels
    into the step scratch and the per-unit kernel only scans. Results must not depend on that choice. bf16 rows go
    through ONE launch of the tensor-core kernel as two row ranges (query rows, key rows), here also with row counts
    that end inside a 128-row tile; fp32 rows go through the CUDA-core kernel, one launch per range."""
    w = wl.CONFIGS["throughput_batch"].scaled(batch=batch, budget_lo=40, budget_hi=64, prompt_factor=1, decode_steps=5,
                                               dtype=dtype)
    case = Case(w)
    case.prefill()
    case.compare_state()
    case.decode(5)


@pytest.mark.parametrize("b", [4, 8, 16, 24, 32, 64])
def test_hash_dimension_sweep(b):
    """The hash widths of the paper's ablation (Section 4.7, Table 9), 4 and 24 bits included: prefill then decode."""
    w = PARITY_CASES["llama3_8b_gqa"].scaled(batch=2, prompt_len=640, budget=257, decode_steps=12, hash_bits=b)
    case = Case(w)
    case.prefill()
    case.compare_state()
    case.decode(12, check_every=4)
