"""Helpers for the GPU-vs-oracle parity tests: same seeded inputs to both sides, staged comparison.

Stage H: device hash codes against the oracle's Eq. 2 codes; a bit may differ only where the oracle's
         fp64 projection is within 1e-5 * |x| * |w| of zero (the oracle's `fragile` mask).
Stage D: the oracle replays Algorithm 1 on the DEVICE's codes, so every integer result (distances /
         scores, victims, evicted positions, pos table, code table, K/V slot bytes) must match bit for bit.
"""
import numpy as np
import torch

import oracle
from paper_2412_16187_b200 import HashEvictCache, hash_keys
from paper_2412_16187_b200 import workloads as wl


def to_dev(a: np.ndarray, w) -> torch.Tensor:
    t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()
    return t.view(torch.bfloat16) if a.dtype == np.uint16 else t


def codes_np(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def torch_dtype(w):
    return torch.bfloat16 if w.dtype == "bf16" else torch.float32


def raw_np(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> numpy with the generator's storage type (bf16 as uint16 bit patterns)."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def check_hash_stage(x_np: np.ndarray, W: np.ndarray, dtype: str, gpu_codes: np.ndarray):
    """Stage H. Returns (mismatching bits, fragile bits) after asserting every mismatch is fragile."""
    ref, fragile = oracle.hash_rows(np.ascontiguousarray(x_np.reshape(-1, x_np.shape[-1])), W, dtype, want_fragile=True)
    diff = ref ^ gpu_codes.reshape(ref.shape)
    bad = diff & ~fragile
    assert not bad.any(), f"{int(np.count_nonzero(bad))} code words differ outside the fragile set"
    popc = lambda a: int(np.unpackbits(a.view(np.uint8)).sum())
    return popc(diff), popc(fragile)


class Case:
    """One workload resident on both sides."""

    def __init__(self, w, write_scores=True, packed_codes=False, early_inputs=False):
        self.w = w
        self.W = wl.gen_W(w)
        self.plen = w.prompt_lens()
        Nmax = w.max_prompt_len
        self.K = wl.gen_tokens(w, "k", 0, w.n_seq, 0, Nmax)
        self.Q = wl.gen_tokens(w, "q", 0, w.n_seq, 0, Nmax)
        self.V = wl.gen_tokens(w, "v", 0, w.n_seq, 0, Nmax)
        self.gpu = HashEvictCache(w.n_seq, w.n_kv_heads, w.group_size, w.head_dim, w.hash_bits, w.budgets(),
                                  torch.from_numpy(self.W), dtype=torch_dtype(w), n_sink=w.n_sink, n_recent=w.n_recent,
                                  write_scores=write_scores, packed_codes=packed_codes, early_inputs=early_inputs)
        self.orc = oracle.OracleCache(w.n_seq, w.n_kv_heads, w.group_size, w.head_dim, w.hash_bits, self.gpu.Cmax,
                                      w.budgets(), w.dtype, n_sink=w.n_sink, n_recent=w.n_recent, threads=8)
        self.dK, self.dQ, self.dV = to_dev(self.K, w), to_dev(self.Q, w), to_dev(self.V, w)
        self.dplen = torch.from_numpy(self.plen).cuda()

    def compare_state(self, what=("codes", "pos", "fill", "next_pos", "scores", "k_cache", "v_cache")):
        g, o = self.gpu, self.orc
        torch.cuda.synchronize()
        for name in what:
            got = getattr(g, name)
            got = codes_np(got) if name == "codes" else raw_np(got)
            want = getattr(o, name)
            if name in ("k_cache", "v_cache"):
                # only valid slots hold defined rows
                fill = o.fill
                for s in range(o.B):
                    for h in range(o.H):
                        f = int(fill[s, h])
                        assert np.array_equal(got[s, h, :f], want[s, h, :f]), f"{name} differs at unit ({s},{h})"
            else:
                assert np.array_equal(got, want), f"{name} differs ({int(np.count_nonzero(got != want))} entries)"

    def prefill(self):
        """he_prefill_compress on the device, then the oracle on the device's prompt codes (stage D)."""
        w = self.w
        Nmax = w.max_prompt_len
        self.gpu.prefill_compress(self.dQ, self.dK, self.dV, self.dplen)
        torch.cuda.synchronize()
        kc, qc = self.gpu.prompt_codes(Nmax)
        kc, qc = codes_np(kc).copy(), codes_np(qc).copy()
        # stage H on every prompt key and on the queries that were hashed (t >= C_s)
        flips = fragile = 0
        for s in range(w.n_seq):
            N, C = int(self.plen[s]), int(w.budgets()[s])
            f, g = check_hash_stage(self.K[s, :, :N], self.W, w.dtype, kc[s, :, :N])
            flips, fragile = flips + f, fragile + g
            if N > C:
                qs = self.Q[s, :, C:N].reshape(w.n_kv_heads, w.group_size, N - C, w.head_dim).transpose(0, 2, 1, 3)
                f, g = check_hash_stage(qs, self.W, w.dtype, qc[s, :, C:N])
                flips, fragile = flips + f, fragile + g
            qc[s, :, :min(C, N)] = 0  # never read by either side
            kc[s, :, N:] = 0
            qc[s, :, N:] = 0
        self.orc.prefill_codes(kc, qc, self.K, self.V, self.plen)
        return flips, fragile

    def decode(self, steps, check_every=1):
        w = self.w
        dq = wl.gen_decode_inputs(w, "q", 0, steps)
        dk = wl.gen_decode_inputs(w, "k", 0, steps)
        dv = wl.gen_decode_inputs(w, "v", 0, steps)
        gq, gk, gv = to_dev(dq, w), to_dev(dk, w), to_dev(dv, w)
        B, H, G, Wd = w.n_seq, w.n_kv_heads, w.group_size, self.gpu.Wd
        victim = torch.empty((B, H), dtype=torch.int32, device="cuda")
        evicted = torch.empty((B, H), dtype=torch.int32, device="cuda")
        qcodes = torch.empty((B, H * G, Wd), dtype=torch.int32, device="cuda")
        flips = fragile = 0
        for i in range(steps):
            self.gpu.decode_step(gq[i], gk[i], gv[i], victim, evicted, qcodes)
            torch.cuda.synchronize()
            vic = victim.cpu().numpy()
            qc = codes_np(qcodes)
            gcodes = codes_np(self.gpu.codes)
            kc = np.take_along_axis(gcodes, vic[:, :, None, None].astype(np.int64), axis=2)[:, :, 0, :]
            f, g = check_hash_stage(dq[i], self.W, w.dtype, qc)
            flips, fragile = flips + f, fragile + g
            f, g = check_hash_stage(dk[i], self.W, w.dtype, kc)
            flips, fragile = flips + f, fragile + g
            ovic, oev = self.orc.step_codes(qc, kc, dk[i], dv[i])
            assert np.array_equal(vic, ovic), f"victims differ at decode step {i}"
            assert np.array_equal(evicted.cpu().numpy(), oev), f"evicted positions differ at decode step {i}"
            if (i + 1) % check_every == 0 or i == steps - 1:
                self.compare_state(("codes", "pos", "fill", "next_pos", "scores"))
        self.compare_state()
        return flips, fragile
