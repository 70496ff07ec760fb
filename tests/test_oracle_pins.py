"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without the oracle's own formulas.

Each test names the passage it pins. The brute-force reference here works on unpacked {0,1}
arrays with bit-by-bit loops, so a mistake in the oracle's packing, popcount, GQA sum,
tie-break or overwrite shows up as a disagreement.
"""
import itertools
import math

import numpy as np
import pytest

import oracle
from paper_2412_16187_b200 import workloads as wl


def unpack(codes, b):
    """[..., Wd] uint32 -> [..., b] array of 0/1, bit i = column i (LSB first)."""
    codes = np.asarray(codes, dtype=np.uint32)
    bits = [(codes[..., i // 32] >> np.uint32(i % 32)) & np.uint32(1) for i in range(b)]
    return np.stack(bits, axis=-1).astype(np.int64)


def pack(bits):
    bits = np.asarray(bits)
    b = bits.shape[-1]
    out = np.zeros(bits.shape[:-1] + ((b + 31) // 32,), dtype=np.uint32)
    for i in range(b):
        out[..., i // 32] |= (bits[..., i].astype(np.uint32) << np.uint32(i % 32))
    return out


# ---------------------------------------------------------------- Eq. 2: h(x) = sgn(Rx)

@pytest.mark.parametrize("dtype,d,b", [("f32", 64, 8), ("bf16", 128, 32), ("bf16", 128, 64), ("f32", 40, 24), ("bf16", 128, 16)])
def test_hash_matches_library_matmul(dtype, d, b):
    rng = np.random.default_rng(1)
    W = rng.standard_normal((d, b)).astype(np.float32)
    x32 = rng.standard_normal((257, d)).astype(np.float32)
    if dtype == "bf16":
        x = (x32.view(np.uint32) >> 16).astype(np.uint16)  # truncation is fine: any bf16 pattern is a valid input
        xd = wl.bf16_to_f32(x).astype(np.float64)
    else:
        x, xd = x32, x32.astype(np.float64)
    codes, fragile, proj = oracle.hash_rows(x, W, dtype, want_fragile=True, want_proj=True)
    ref = xd @ W.astype(np.float64)  # library routine, fp64
    np.testing.assert_allclose(proj, ref, rtol=1e-12, atol=1e-12)
    safe = np.abs(ref) > 1e-9
    assert np.array_equal(unpack(codes, b)[safe], (ref >= 0).astype(np.int64)[safe])
    # bits beyond b stay zero
    if b % 32:
        assert np.all(codes[:, -1] >> np.uint32(b % 32) == 0)
    # fragile mask is the stated rule
    bound = 1e-5 * np.linalg.norm(xd, axis=1)[:, None] * np.linalg.norm(W.astype(np.float64), axis=0)[None, :]
    assert np.array_equal(unpack(fragile, b), (np.abs(ref) < bound).astype(np.int64))


def test_hash_bit_order_and_operand_orientation():
    # x = e_3 picks row 3 of W; column i of W decides bit i. A transposed W or MSB-first packing fails.
    d, b = 48, 40
    W = np.zeros((d, b), dtype=np.float32)
    on = {0, 1, 5, 31, 32, 39}
    for i in range(b):
        W[3, i] = 1.0 if i in on else -1.0
    W[7, :] = 123.0  # must not matter: x_7 = 0
    x = np.zeros((1, d), dtype=np.float32)
    x[0, 3] = 2.5
    codes = oracle.hash_rows(x, W, "f32")
    expect = [sum(1 << i for i in on if i < 32), sum(1 << (i - 32) for i in on if i >= 32)]
    assert codes[0].tolist() == expect


def test_hash_sign_conventions():
    rng = np.random.default_rng(2)
    d, b = 64, 48
    W = rng.standard_normal((d, b)).astype(np.float32)
    x = rng.standard_normal((50, d)).astype(np.float32)
    c = oracle.hash_rows(x, W, "f32")
    # scale invariance: h(a x) = h(x) for a > 0 (powers of two keep the products exact)
    assert np.array_equal(oracle.hash_rows((x * 4.0).astype(np.float32), W, "f32"), c)
    assert np.array_equal(oracle.hash_rows((x * 0.125).astype(np.float32), W, "f32"), c)
    # antipodal: every bit flips (no projection is exactly 0 here), so d_H(h(x), h(-x)) = b
    cneg = oracle.hash_rows(-x, W, "f32")
    assert np.all((unpack(c, b) ^ unpack(cneg, b)) == 1)
    # sgn(0) = 1: the zero vector hashes to all ones, -0.0 too
    z = np.zeros((2, d), dtype=np.float32)
    z[1] = -0.0
    cz = oracle.hash_rows(z, W, "f32")
    assert np.all(unpack(cz, b) == 1) and cz[0].tolist() == [0xFFFFFFFF, 0xFFFF]


# ---------------------------------------------------------------- Eq. 3: E[d_H]/b = theta/pi

@pytest.mark.parametrize("theta", [0.0, math.pi / 6, math.pi / 3, math.pi / 2, 2 * math.pi / 3, math.pi])
def test_simhash_expectation(theta):
    d, b, trials = 32, 64, 320  # 20480 independent hyperplanes
    rng = np.random.default_rng(7)
    x = np.zeros((1, d), dtype=np.float32)
    y = np.zeros((1, d), dtype=np.float32)
    x[0, 0] = 1.0
    y[0, 0], y[0, 1] = math.cos(theta), math.sin(theta)
    tot = 0
    for _ in range(trials):
        W = rng.standard_normal((d, b)).astype(np.float32)
        tot += int((unpack(oracle.hash_rows(x, W, "f32"), b) ^ unpack(oracle.hash_rows(y, W, "f32"), b)).sum())
    n = trials * b
    p = theta / math.pi
    sigma = math.sqrt(max(p * (1 - p), 1e-12) / n)
    assert abs(tot / n - p) <= 4 * sigma + 1e-9


# ---------------------------------------------------------------- Eq. 5 / Eq. 6 / Algorithm 1: brute force

def brute_victim(table_bits, q_bits, pos, t, n_sink, n_recent):
    """table_bits [C][b], q_bits [G][b] as 0/1 lists. Returns (victim, distances)."""
    C = len(table_bits)
    D = []
    for j in range(C):
        dist = 0
        for g in range(len(q_bits)):
            for i in range(len(q_bits[g])):
                if table_bits[j][i] != q_bits[g][i]:
                    dist += 1
        D.append(dist)
    order = [j for j in range(C) if pos[j] >= n_sink and pos[j] < t - n_recent] or list(range(C))
    worst = max(D[j] for j in order)
    return min(j for j in order if D[j] == worst), D


def make_full_cache(C, b, G, table_codes, n_sink=0, n_recent=0, d=8):
    oc = oracle.OracleCache(1, 1, G, d, b, C, [C], "f32", n_sink=n_sink, n_recent=n_recent)
    oc.codes[0, 0] = table_codes
    oc.pos[0, 0] = np.arange(C)
    oc.fill[:] = C
    oc.next_pos[:] = C
    return oc


def test_victim_exhaustive_c3_b3():
    C, b = 3, 3
    k = np.ones((1, 1, 8), dtype=np.float32)
    for table in itertools.product(range(8), repeat=C):
        for qv in range(8):
            tb = [[(c >> i) & 1 for i in range(b)] for c in table]
            qb = [[(qv >> i) & 1 for i in range(b)]]
            oc = make_full_cache(C, b, 1, np.array(table, dtype=np.uint32).reshape(C, 1))
            victim, evicted = oc.step_codes(np.array([[[qv]]]), np.array([[[5]]]), k, k)
            want, D = brute_victim(tb, qb, list(range(C)), C, 0, 0)
            assert victim[0, 0] == want and evicted[0, 0] == want
            assert oc.scores[0, 0].tolist() == [-float(x) for x in D]
            assert oc.codes[0, 0, want, 0] == 5 and oc.pos[0, 0, want] == C


@pytest.mark.parametrize("C,b,G", [(8, 8, 1), (8, 8, 2), (5, 40, 2), (7, 64, 4), (6, 33, 3)])
def test_victim_brute_force_random_tables(C, b, G):
    rng = np.random.default_rng(C * 100 + b + G)
    k = np.ones((1, 1, 8), dtype=np.float32)
    queries = itertools.product(range(256), repeat=G) if b == 8 and G == 1 else None
    for trial in range(256 if queries is None else 1):
        tb = rng.integers(0, 2, size=(C, b))
        # few distinct rows so that ties are common
        tb[rng.integers(0, C)] = tb[rng.integers(0, C)]
        qsets = [rng.integers(0, 2, size=(G, b)) for _ in range(4)] if queries is None else \
            [np.array([[(qv >> i) & 1 for i in range(b)] for qv in qs]) for qs in queries]
        for qb in qsets:
            oc = make_full_cache(C, b, G, pack(tb))
            victim, _ = oc.step_codes(pack(qb)[None], pack(rng.integers(0, 2, size=(1, 1, b))), k, k)
            want, D = brute_victim(tb.tolist(), qb.tolist(), list(range(C)), C, 0, 0)
            assert victim[0, 0] == want
            assert oc.scores[0, 0].tolist() == [-float(x) for x in D]


def test_victim_with_protected_tokens():
    C, b, G = 12, 16, 2
    rng = np.random.default_rng(11)
    k = np.ones((1, 1, 8), dtype=np.float32)
    for trial in range(300):
        n_sink, n_recent = int(rng.integers(0, 4)), int(rng.integers(0, 4))
        tb = rng.integers(0, 2, size=(C, b))
        qb = rng.integers(0, 2, size=(G, b))
        pos = rng.permutation(40)[:C]
        t = 40
        oc = make_full_cache(C, b, G, pack(tb), n_sink=n_sink, n_recent=n_recent)
        oc.pos[0, 0] = pos
        oc.next_pos[:] = t
        victim, evicted = oc.step_codes(pack(qb)[None], pack(rng.integers(0, 2, size=(1, 1, b))), k, k)
        want, _ = brute_victim(tb.tolist(), qb.tolist(), pos.tolist(), t, n_sink, n_recent)
        assert victim[0, 0] == want and evicted[0, 0] == pos[want]


# ---------------------------------------------------------------- Section 3 state invariants

def run_tiny(n_sink=0, n_recent=0, G=1, b=8, C=16, N=40, T=24, heads=2, d=16, dtype="f32", seed=0):
    w = wl.Workload("t", seed, 1, 2, heads, G, d, dtype, b, N, C, T, wl.KIND_IID, n_sink=n_sink, n_recent=n_recent)
    W = wl.gen_W(w)
    K = wl.gen_tokens(w, "k", 0, 2, 0, N + T)
    Q = wl.gen_tokens(w, "q", 0, 2, 0, N + T)
    V = wl.gen_tokens(w, "v", 0, 2, 0, N + T)
    oc = oracle.OracleCache(2, heads, G, d, b, C, [C, C - 3], dtype, n_sink=n_sink, n_recent=n_recent)
    return w, W, K, Q, V, oc


@pytest.mark.parametrize("n_sink,n_recent,G,b,dtype", [(0, 0, 1, 8, "f32"), (4, 10, 1, 8, "f32"), (2, 3, 4, 40, "bf16"), (0, 5, 2, 64, "bf16")])
def test_state_invariants_every_step(n_sink, n_recent, G, b, dtype):
    w, W, K, Q, V, oc = run_tiny(n_sink, n_recent, G, b, dtype=dtype)
    budgets = oc.budget
    for t in range(K.shape[2]):
        q = np.ascontiguousarray(Q[:, :, t])
        k = np.ascontiguousarray(K[:, :, t])
        v = np.ascontiguousarray(V[:, :, t])
        victim, evicted, qc, kc = oc.step(W, q, k, v)
        for s in range(2):
            C = int(budgets[s])
            for h in range(w.n_kv_heads):
                fill = oc.fill[s, h]
                assert fill == min(t + 1, C)  # constant budget (Section 3, "Complexity")
                assert oc.next_pos[s, h] == t + 1
                slot = victim[s, h]
                assert oc.pos[s, h, slot] == t  # the newest token is resident (Algorithm 1 lines 3-5)
                pos = oc.pos[s, h, :fill]
                assert len(set(pos.tolist())) == fill and np.all(oc.pos[s, h, fill:] == -1)
                # slot contents belong to the token the slot says it holds; H_t = h(K_t)
                assert np.array_equal(oc.k_cache[s, h, :fill], K[s, h, pos])
                assert np.array_equal(oc.v_cache[s, h, :fill], V[s, h, pos])
                assert np.array_equal(oc.codes[s, h, :fill], oracle.hash_rows(np.ascontiguousarray(K[s, h, pos]), W, dtype))
                if t + 1 > C:  # protected tokens present once the cache is full and protection is satisfiable
                    if C > n_sink + n_recent + 1:
                        present = set(pos.tolist())
                        assert all(p in present for p in range(min(n_sink, C)))
                        assert all(p in present for p in range(t - n_recent, t + 1))
                if t >= C:
                    assert evicted[s, h] >= 0 and evicted[s, h] not in set(pos.tolist())
                else:
                    assert evicted[s, h] == -1 and slot == t


def test_prefill_equals_reset_plus_steps_and_short_prompts():
    w, W, K, Q, V, oc = run_tiny(1, 2, 2, 24, C=16, N=40, T=0, dtype="bf16")
    plen = np.array([40, 9], dtype=np.int32)  # second prompt is shorter than its budget (13)
    kc, qc = oc.prefill(W, Q, K, V, plen, want_codes=True)
    # step-by-step replay, one sequence at a time (sequences are independent)
    for s in range(2):
        o1 = oracle.OracleCache(1, w.n_kv_heads, 2, w.head_dim, 24, 16, oc.budget[s:s + 1], "bf16", n_sink=1, n_recent=2)
        for t in range(int(plen[s])):
            o1.step(W, np.ascontiguousarray(Q[s:s + 1, :, t]), np.ascontiguousarray(K[s:s + 1, :, t]),
                    np.ascontiguousarray(V[s:s + 1, :, t]))
        for name in ("k_cache", "v_cache", "codes", "scores", "pos", "fill", "next_pos"):
            assert np.array_equal(getattr(o1, name)[0], getattr(oc, name)[s]), name
    # short prompt: identity placement, nothing evicted
    assert oc.fill[1].tolist() == [9] * w.n_kv_heads
    assert np.array_equal(oc.pos[1, :, :9], np.tile(np.arange(9), (w.n_kv_heads, 1)))
    assert np.array_equal(oc.k_cache[1, :, :9], K[1, :, :9])
    # prefill on its own codes == prefill from embeddings
    oc3 = oracle.OracleCache(2, w.n_kv_heads, 2, w.head_dim, 24, 16, oc.budget, "bf16", n_sink=1, n_recent=2)
    oc3.prefill_codes(kc, qc, K, V, plen)
    for name in ("k_cache", "v_cache", "codes", "scores", "pos", "fill", "next_pos"):
        assert np.array_equal(getattr(oc3, name), getattr(oc, name)), name


def test_threads_do_not_change_results():
    w, W, K, Q, V, oc = run_tiny(0, 0, 2, 16)
    oc.prefill(W, Q, K, V, np.array([64, 64], dtype=np.int32))
    oc4 = oracle.OracleCache(2, w.n_kv_heads, 2, w.head_dim, 16, 16, oc.budget, "f32", threads=4)
    oc4.prefill(W, Q, K, V, np.array([64, 64], dtype=np.int32))
    for name in ("k_cache", "codes", "scores", "pos", "fill"):
        assert np.array_equal(getattr(oc4, name), getattr(oc, name))


# ---------------------------------------------------------------- Section 4.7: hash-table storage

def test_hash_table_storage_closed_form():
    # Llama-3-70B example: 80 layers, 8 KV heads, sequence 8192, batch 8, 50 % budget -> 80 MB at 32 bits,
    # i.e. b/8 bytes per slot per KV head. One layer of that shape in the oracle's packed layout:
    oc = oracle.OracleCache(8, 8, 1, 8, 32, 4096, [4096] * 8, "bf16")
    assert oc.codes.nbytes * 80 == 80 * 2 ** 20
    # the paper's 8- and 16-bit figures (20 MB, 40 MB) follow from the same b/8 bytes per slot
    slots = 80 * 8 * 8 * 4096
    assert [slots * b // 8 // 2 ** 20 for b in (8, 16, 32)] == [20, 40, 80]


# ---------------------------------------------------------------- Eq. 1 on the compressed cache (Algorithm 1 line 6)

def test_attend_matches_library_softmax_attention():
    import torch

    w, W, K, Q, V, oc = run_tiny(0, 0, 4, 16, C=16, N=40, T=0, dtype="bf16")
    oc.prefill(W, Q, K, V, np.array([40, 11], dtype=np.int32))  # second sequence: 11 of 13 slots filled
    q = np.ascontiguousarray(Q[:, :, 5])
    out = oc.attend(q)
    Kc, Vc, qd = (torch.from_numpy(wl.as_f64(w, a)) for a in (oc.k_cache, oc.v_cache, q))
    for s in range(2):
        for h in range(w.n_kv_heads):
            f = int(oc.fill[s, h])
            for g in range(4):
                qq = qd[s, h * 4 + g]
                p = torch.softmax((Kc[s, h, :f] @ qq) / np.sqrt(w.head_dim), dim=0)  # library softmax, fp64
                np.testing.assert_allclose(out[s, h * 4 + g], (p[:, None] * Vc[s, h, :f]).sum(0).numpy(), rtol=1e-12, atol=1e-12)


def test_attend_special_cases():
    d = 16
    oc = oracle.OracleCache(1, 1, 2, d, 8, 8, [8], "f32")
    rng = np.random.default_rng(5)
    q = rng.standard_normal((1, 2, d)).astype(np.float32)
    assert not oc.attend(q).any()  # empty cache
    oc.fill[:] = 1
    oc.k_cache[0, 0, 0] = rng.standard_normal(d)
    oc.v_cache[0, 0, 0] = np.arange(d)
    np.testing.assert_allclose(oc.attend(q)[0, 1], np.arange(d), rtol=1e-15)  # one slot: its V row, whatever q is
    oc.fill[:] = 5
    oc.k_cache[0, 0, :5] = oc.k_cache[0, 0, 0]  # equal keys: uniform weights, the mean of V
    oc.v_cache[0, 0, :5] = rng.standard_normal((5, d))
    np.testing.assert_allclose(oc.attend(q)[0, 0], oc.v_cache[0, 0, :5].astype(np.float64).mean(0), rtol=1e-12, atol=1e-12)
    oc.k_cache[0, 0, :5] = rng.standard_normal((5, d))
    a = oc.attend(q).copy()
    perm = np.array([3, 1, 4, 0, 2])
    oc.k_cache[0, 0, :5] = oc.k_cache[0, 0, perm]
    oc.v_cache[0, 0, :5] = oc.v_cache[0, 0, perm]
    np.testing.assert_allclose(oc.attend(q), a, rtol=1e-12, atol=1e-13)  # the slot order does not matter


# ---------------------------------------------------------------- one-shot averaged-Hamming ranking (Appendix C)

def test_oneshot_worked_example():
    # b = 2, G = 1, three tokens, budget 2. Key codes 00, 11, 01; query codes (of tokens 1, 2) 01, 10.
    # S_0 = |00^01| + |00^10| = 2 over n = 2 -> 1; S_1 = |11^10| = 1 over n = 1 -> 1; token 2 has no later query -> 0.
    # Order: token 2, then the tie at 1 by index: 0, 1. Kept: {0, 2}, stored in token order.
    oc = oracle.OracleCache(1, 1, 1, 8, 2, 4, [2], "f32")
    kc = np.array([0b00, 0b11, 0b01], dtype=np.uint32).reshape(1, 1, 3, 1)
    qc = np.array([0b11, 0b01, 0b10], dtype=np.uint32).reshape(1, 1, 3, 1, 1)  # token 0's query is never used
    k = np.arange(24, dtype=np.float32).reshape(1, 1, 3, 8)
    v = -k
    sums = oc.oneshot_codes(kc, qc, k, v, [3], want_sums=True)
    assert sums[0, 0].tolist() == [2, 1, 0]
    assert oc.pos[0, 0].tolist() == [0, 2, -1, -1] and oc.fill[0, 0] == 2 and oc.next_pos[0, 0] == 3
    assert oc.scores[0, 0].tolist() == [-1.0, 0.0, 0.0, 0.0]
    assert np.array_equal(oc.k_cache[0, 0, 1], k[0, 0, 2]) and np.array_equal(oc.v_cache[0, 0, 0], v[0, 0, 0])
    assert oc.codes[0, 0, :2, 0].tolist() == [0b00, 0b01]


@pytest.mark.parametrize("G,b,n_sink,n_recent", [(1, 8, 0, 0), (4, 40, 0, 0), (2, 64, 3, 5), (3, 16, 0, 2)])
def test_oneshot_against_per_bit_counts_and_exact_fractions(G, b, n_sink, n_recent):
    from fractions import Fraction

    rng = np.random.default_rng(11 + G)
    B, H, N, C, d = 2, 2, 57, 20, 8
    Wd = oracle.words(b)
    mask = [(1 << min(32, b - 32 * w)) - 1 for w in range(Wd)]
    kc = rng.integers(0, 2**32, size=(B, H, N, Wd), dtype=np.uint64).astype(np.uint32) & np.array(mask, dtype=np.uint32)
    qc = rng.integers(0, 2**32, size=(B, H, N, G, Wd), dtype=np.uint64).astype(np.uint32) & np.array(mask, dtype=np.uint32)
    kc[0, 0, 5:9] = kc[0, 0, 4]  # equal keys next to each other: equal sums only if their later queries agree
    qc[1, 1, 30:] = qc[1, 1, 29]  # a constant tail of queries: many equal averages
    plen = np.array([N, 13], dtype=np.int32)  # the second sequence is shorter than its budget
    oc = oracle.OracleCache(B, H, G, d, b, C, [C, C - 3], "f32", n_sink=n_sink, n_recent=n_recent)
    k = rng.standard_normal((B, H, N, d)).astype(np.float32)
    v = rng.standard_normal((B, H, N, d)).astype(np.float32)
    sums = oc.oneshot_codes(kc, qc, k, v, plen, want_sums=True)
    for s in range(B):
        n_tok, cap = int(plen[s]), int(oc.budget[s])
        for h in range(H):
            kb = unpack(kc[s, h, :n_tok], b).astype(np.int64)          # [N, b]
            qb = unpack(qc[s, h, :n_tok].reshape(n_tok * G, Wd), b).reshape(n_tok, G, b).astype(np.int64).sum(1)  # ones per bit
            later = np.concatenate([np.cumsum(qb[::-1], axis=0)[::-1][1:], np.zeros((1, b), dtype=np.int64)])  # tokens j > i
            m = (n_tok - 1 - np.arange(n_tok))[:, None] * G
            want = np.where(kb == 1, m - later, later).sum(1)  # a set key bit differs from the zeros, a clear one from the ones
            assert np.array_equal(sums[s, h, :n_tok], want)
            prot = [i for i in range(n_tok) if i < n_sink or i >= n_tok - n_recent]
            rest = sorted((i for i in range(n_tok) if i not in prot),
                          key=lambda i: (Fraction(int(want[i]), max(1, n_tok - 1 - i)), i))
            keep = sorted((prot + rest)[:min(n_tok, cap)])
            fill = int(oc.fill[s, h])
            assert fill == len(keep) and oc.pos[s, h, :fill].tolist() == keep and np.all(oc.pos[s, h, fill:] == -1)
            assert oc.next_pos[s, h] == n_tok
            for sl, t in enumerate(keep):
                assert np.array_equal(oc.codes[s, h, sl], kc[s, h, t]) and np.array_equal(oc.k_cache[s, h, sl], k[s, h, t])
                n = n_tok - 1 - t
                assert oc.scores[s, h, sl] == (-(np.float32(want[t]) / np.float32(n)) if n > 0 else 0.0)


def test_oneshot_special_cases():
    b, G, N, C = 16, 2, 12, 5
    oc = oracle.OracleCache(1, 1, G, 8, b, C, [C], "f32")
    k = np.zeros((1, 1, N, 8), dtype=np.float32)
    kc = np.full((1, 1, N, 1), 0x1234, dtype=np.uint32)
    same = np.full((1, 1, N, G, 1), 0x1234, dtype=np.uint32)
    sums = oc.oneshot_codes(kc, same, k, k, [N], want_sums=True)
    assert not sums.any() and oc.pos[0, 0].tolist() == [0, 1, 2, 3, 4]  # all averages equal: the lowest indices stay
    sums = oc.oneshot_codes(kc, same ^ np.uint32(0xFFFF), k, k, [N], want_sums=True)
    assert sums[0, 0].tolist() == [G * b * (N - 1 - i) for i in range(N)]  # complementary codes: every bit differs
    # average G*b for all but the last token (0): the last token first, then the lowest indices
    assert oc.pos[0, 0].tolist() == [0, 1, 2, 3, N - 1]


# ---------------------------------------------------------------- L2-norm ranking and attention loss (comparison policy, Section 4.6)

def test_l2_ranking_norms_order_and_state():
    rng = np.random.default_rng(3)
    B, H, N, C, d, b = 2, 2, 41, 12, 16, 8
    k = rng.standard_normal((B, H, N, d)).astype(np.float32)
    v = rng.standard_normal((B, H, N, d)).astype(np.float32)
    k[0, 0, 7] = k[0, 0, 3]  # equal norms: the lower index ranks first
    k[1, 1, :, :] *= np.linspace(2.0, 0.5, N, dtype=np.float32)[:, None]  # norms fall with the position: the newest stay
    kc = rng.integers(0, 256, size=(B, H, N, 1), dtype=np.uint32)
    plen = np.array([N, 9], dtype=np.int32)
    for n_sink, n_recent in [(0, 0), (2, 3)]:
        oc = oracle.OracleCache(B, H, 1, d, b, C, [C, C], "f32", n_sink=n_sink, n_recent=n_recent)
        norms = oc.oneshot_l2(kc, k, v, plen, want_norms=True)
        for s in range(B):
            n_tok = int(plen[s])
            for h in range(H):
                exact = (k[s, h, :n_tok].astype(np.float64) ** 2).sum(1)
                np.testing.assert_allclose(norms[s, h, :n_tok], exact, rtol=2e-6)  # fp32 chain of 16 terms
                prot = [i for i in range(n_tok) if i < n_sink or i >= n_tok - n_recent]
                rest = sorted((i for i in range(n_tok) if i not in prot), key=lambda i: (norms[s, h, i], i))
                keep = sorted((prot + rest)[:min(n_tok, C)])
                fill = int(oc.fill[s, h])
                assert oc.pos[s, h, :fill].tolist() == keep and oc.next_pos[s, h] == n_tok
                for sl, t in enumerate(keep):
                    assert np.array_equal(oc.k_cache[s, h, sl], k[s, h, t]) and oc.codes[s, h, sl, 0] == kc[s, h, t, 0]
                    assert oc.scores[s, h, sl] == -norms[s, h, t]
        if n_sink == 0:
            assert oc.pos[1, 1, :9].tolist() == list(range(9))  # short prompt: everything stays
    # the summation order is part of the definition: 2^12 squared, then sixteen ones, in fp32
    x = np.zeros((1, 1, 2, 32), dtype=np.float32)
    x[0, 0, 0, 0] = 4096.0
    x[0, 0, 0, 1:17] = 1.0   # ascending chain: each +1 is lost against 2^24
    x[0, 0, 1, 16] = 4096.0
    x[0, 0, 1, 0:16] = 1.0   # the ones first: 16, then + 2^24 is exact
    oc = oracle.OracleCache(1, 1, 1, 32, 8, 4, [4], "f32")
    nn = oc.oneshot_l2(np.zeros((1, 1, 2, 1), dtype=np.uint32), x, x, [2], want_norms=True)
    assert nn[0, 0].tolist() == [2.0 ** 24, 2.0 ** 24 + 16.0]


def test_attention_loss_closed_forms_and_library_softmax():
    import torch

    w, W, K, Q, V, oc = run_tiny(0, 0, 2, 16, C=16, N=40, T=0, dtype="bf16")
    q = np.ascontiguousarray(Q[:, :, 39])
    oc.prefill(W, Q, K, V, np.array([40, 11], dtype=np.int32))
    loss = oc.attention_loss(q, K)
    Kd, qd = torch.from_numpy(wl.as_f64(w, K)), torch.from_numpy(wl.as_f64(w, q))
    for s in range(2):
        n = int(oc.next_pos[s, 0])
        for h in range(w.n_kv_heads):
            fill = int(oc.fill[s, h])
            for g in range(2):
                a = torch.softmax((Kd[s, h, :n] @ qd[s, h * 2 + g]) / np.sqrt(w.head_dim), dim=0).numpy()
                want = 1.0 - a[oc.pos[s, h, :fill]].sum()
                assert abs(loss[s, h * 2 + g] - want) < 1e-12
    assert np.all(np.abs(loss[1]) < 1e-12)  # the second prompt fits its budget: nothing was dropped
    assert np.all(loss[0] > 0) and np.all(loss[0] < 1)
    # equal keys: uniform attention, the loss is the dropped fraction
    oc2 = oracle.OracleCache(1, 1, 1, 8, 8, 4, [4], "f32")
    kk = np.ones((1, 1, 10, 8), dtype=np.float32)
    oc2.oneshot_l2(np.zeros((1, 1, 10, 1), dtype=np.uint32), kk, kk, [10])
    out = oc2.attention_loss(np.full((1, 1, 8), 0.3, dtype=np.float32), kk)
    assert abs(out[0, 0] - 0.6) < 1e-12
    # one key carries all the attention: loss 0 if it is cached, 1 if it is not
    kk[0, 0, 2] = 50.0   # huge norm: the L2 ranking drops it first
    oc2.oneshot_l2(np.zeros((1, 1, 10, 1), dtype=np.uint32), kk, kk, [10])
    assert 2 not in oc2.pos[0, 0].tolist()
    assert oc2.attention_loss(np.ones((1, 1, 8), dtype=np.float32), kk)[0, 0] > 1 - 1e-12
    # the opposite: a zero key (lowest norm, ranked first) under a query that scores every other key far below it
    kk = np.full((1, 1, 10, 8), 3.0, dtype=np.float32)
    kk[0, 0, 2] = 0.0
    oc2.oneshot_l2(np.zeros((1, 1, 10, 1), dtype=np.uint32), kk, kk, [10])
    assert 2 in oc2.pos[0, 0].tolist()
    out = oc2.attention_loss(-np.ones((1, 1, 8), dtype=np.float32), kk)[0, 0]
    assert 0 < out < 6 * np.exp(-24 / np.sqrt(8)) * 1.01  # six dropped keys, each e^(-24/sqrt 8) of the kept zero key


def test_l2_decode_steps_keep_the_lowest_norms_and_the_newest_token():
    rng = np.random.default_rng(9)
    B, H, d, C, T = 1, 2, 16, 6, 30
    for n_sink, n_recent in [(0, 0), (1, 2)]:
        oc = oracle.OracleCache(B, H, 1, d, 8, C, [C], "f32", n_sink=n_sink, n_recent=n_recent)
        ks = rng.standard_normal((T, B, H, d)).astype(np.float32) * rng.uniform(0.2, 3.0, size=(T, 1, H, 1)).astype(np.float32)
        ks[11] = ks[7]  # equal norms: the lower slot leaves first
        resident = [dict() for _ in range(H)]  # slot -> (token, norm2), replayed in Python
        for t in range(T):
            victim, evicted = oc.step_l2(np.ascontiguousarray(ks[t]), np.ascontiguousarray(-ks[t]))
            for h in range(H):
                n2 = np.float32(0)
                for c in range(d):
                    n2 = np.float32(np.float64(ks[t, 0, h, c]) ** 2 + np.float64(n2))  # one rounding per channel, ascending
                res = resident[h]
                if len(res) < C:
                    slot, gone = len(res), -1
                else:
                    elig = [j for j in res if res[j][0] >= n_sink and res[j][0] < t - n_recent] or list(res)
                    slot = min(elig, key=lambda j: (-res[j][1], j))
                    gone = res[slot][0]
                assert victim[0, h] == slot and evicted[0, h] == gone
                res[slot] = (t, n2)
                assert oc.pos[0, h, slot] == t and oc.scores[0, h, slot] == -n2  # the newest token is always resident
                assert np.array_equal(oc.k_cache[0, h, slot], ks[t, 0, h]) and np.array_equal(oc.v_cache[0, h, slot], -ks[t, 0, h])
        if (n_sink, n_recent) == (0, 0):  # what is left: the newest token and the C - 1 lowest norms before it
            for h in range(H):
                n2 = (ks[:T - 1, 0, h].astype(np.float64) ** 2).sum(1)
                want = set(np.argsort(n2, kind="stable")[:C - 1].tolist()) | {T - 1}
                assert set(oc.pos[0, h].tolist()) == want


def test_prefill_follows_the_strides_of_token_major_inputs():
    """The prompt tensors may be strided views (token-major storage, as a fused QKV projection leaves them; a slice of
    a longer buffer): the oracle must read the same tokens as from contiguous copies. Both the embedding route and the
    code route, with ragged prompts so that a wrong stride lands on another token's row."""
    rng = np.random.default_rng(7)
    B, H, G, d, b, N, C = 2, 3, 2, 16, 12, 40, 9
    W = rng.standard_normal((d, b)).astype(np.float32)
    # token-major storage [B, N + 5, heads, d], seen as [B, heads, N, d] through a transpose and a slice
    Kt = rng.standard_normal((B, N + 5, H, d)).astype(np.float32)
    Vt = rng.standard_normal((B, N + 5, H, d)).astype(np.float32)
    Qt = rng.standard_normal((B, N + 5, H * G, d)).astype(np.float32)
    Kv, Vv, Qv = (x[:, 2:N + 2].transpose(0, 2, 1, 3) for x in (Kt, Vt, Qt))
    assert not Kv.flags.c_contiguous and Kv.strides[2] == H * d * 4
    plen = np.array([N, 23], dtype=np.int32)
    budgets = np.array([C, 7], dtype=np.int32)

    def run(q, k, v):
        oc = oracle.OracleCache(B, H, G, d, b, 12, budgets, "f32", n_sink=1, n_recent=2, threads=2)
        oc.prefill(W, q, k, v, plen)
        return oc

    a = run(Qv, Kv, Vv)
    c = run(np.ascontiguousarray(Qv), np.ascontiguousarray(Kv), np.ascontiguousarray(Vv))
    for name in ("codes", "pos", "fill", "next_pos", "scores", "k_cache", "v_cache"):
        assert np.array_equal(getattr(a, name), getattr(c, name)), name
    # the code route: codes hashed from the contiguous copies, K / V handed over as the strided views
    kc = np.stack([oracle.hash_rows(np.ascontiguousarray(Kv[s]).reshape(-1, d), W, "f32").reshape(H, N, -1) for s in range(B)])
    qc = np.stack([oracle.hash_rows(np.ascontiguousarray(Qv[s]).reshape(-1, d), W, "f32").reshape(H, G, N, -1).transpose(0, 2, 1, 3)
                   for s in range(B)])
    e = oracle.OracleCache(B, H, G, d, b, 12, budgets, "f32", n_sink=1, n_recent=2, threads=2)
    e.prefill_codes(np.ascontiguousarray(kc), np.ascontiguousarray(qc), Kv, Vv, plen)
    for name in ("codes", "pos", "fill", "next_pos", "scores", "k_cache", "v_cache"):
        assert np.array_equal(getattr(e, name), getattr(c, name)), name
    # and the rows really are the tokens the positions name
    for s in range(B):
        for h in range(H):
            for j in range(int(c.fill[s, h])):
                assert np.array_equal(a.k_cache[s, h, j], Kt[s, 2 + c.pos[s, h, j], h])
