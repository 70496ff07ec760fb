"""ctypes loader for the CPU oracle (hashevict_oracle.cpp). TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu_baseline / reference legs may import
this package; the CUDA library and its Python binding never do. Arrays are NumPy; bf16 tensors
are carried as uint16 bit patterns. Each wrapper only marshals arguments: the arithmetic is in
the C++ file, which cites the passages of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hashevict_oracle.cpp")
_LIB = os.path.join(_HERE, "libhe_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 (no CUDA, no code shared with the GPU path)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("batch", "n_kv_heads", "group_size", "head_dim", "hash_bits", "max_budget", "n_sink", "n_recent", "dtype")]


class _Cache(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("k_cache", "v_cache", "codes", "scores", "pos", "budget", "fill", "next_pos")]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        lib.orc_hash.argtypes = [vp, i64, i64, i32, i32, vp, i32, vp, vp, vp]
        lib.orc_reset.argtypes = [vp, vp]
        lib.orc_step_codes.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32]
        lib.orc_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32]
        lib.orc_prefill_codes.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32]
        lib.orc_prefill.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, i32]
        lib.orc_oneshot_codes.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, i32]
        lib.orc_oneshot_codes.restype = None
        lib.orc_oneshot_l2.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp, i32]
        lib.orc_oneshot_l2.restype = None
        lib.orc_step_l2.argtypes = [vp, vp, vp, vp, vp, vp, i32]
        lib.orc_step_l2.restype = None
        lib.orc_attention_loss.argtypes = [vp, vp, vp, vp, vp, vp]
        lib.orc_attention_loss.restype = None
        lib.orc_attend.argtypes = [vp, vp, vp, vp]
        lib.orc_attend.restype = None
        for f in (lib.orc_hash, lib.orc_reset, lib.orc_step_codes, lib.orc_step, lib.orc_prefill_codes, lib.orc_prefill):
            f.restype = None
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data


def words(b: int) -> int:
    return (b + 31) // 32


def hash_rows(x: np.ndarray, W: np.ndarray, dtype: str, want_fragile: bool = False, want_proj: bool = False):
    """Eq. 2 on the rows of x [rows, d] (fp32, or bf16 as uint16). Returns codes [rows, Wd] (+ fragile mask, + fp64 projections)."""
    assert x.ndim == 2 and x.flags.c_contiguous and W.dtype == np.float32 and W.flags.c_contiguous
    rows, d = x.shape
    b = W.shape[1]
    assert W.shape[0] == d
    codes = np.zeros((rows, words(b)), dtype=np.uint32)
    fragile = np.zeros_like(codes) if want_fragile else None
    proj = np.zeros((rows, b), dtype=np.float64) if want_proj else None
    _load().orc_hash(_p(x), rows, d, d, 1 if dtype == "bf16" else 0, _p(W), b, _p(codes), _p(fragile), _p(proj))
    out = (codes,)
    if want_fragile:
        out += (fragile,)
    if want_proj:
        out += (proj,)
    return out if len(out) > 1 else codes


class OracleCache:
    """Host-side cache state with the same array layout as the device library's cache."""

    def __init__(self, batch, n_kv_heads, group_size, head_dim, hash_bits, max_budget, budgets, dtype,
                 n_sink=0, n_recent=0, threads=1):
        self.B, self.H, self.G, self.d, self.b = batch, n_kv_heads, group_size, head_dim, hash_bits
        self.Cmax, self.dtype, self.threads = max_budget, dtype, threads
        self.Wd = words(hash_bits)
        np_dt = np.uint16 if dtype == "bf16" else np.float32
        self.k_cache = np.zeros((batch, n_kv_heads, max_budget, head_dim), dtype=np_dt)
        self.v_cache = np.zeros_like(self.k_cache)
        self.codes = np.zeros((batch, n_kv_heads, max_budget, self.Wd), dtype=np.uint32)
        self.scores = np.zeros((batch, n_kv_heads, max_budget), dtype=np.float32)
        self.pos = np.full((batch, n_kv_heads, max_budget), -1, dtype=np.int32)
        self.budget = np.ascontiguousarray(budgets, dtype=np.int32)
        assert self.budget.shape == (batch,) and int(self.budget.max()) <= max_budget
        self.fill = np.zeros((batch, n_kv_heads), dtype=np.int32)
        self.next_pos = np.zeros((batch, n_kv_heads), dtype=np.int32)
        self._cfg = _Config(batch, n_kv_heads, group_size, head_dim, hash_bits, max_budget, n_sink, n_recent,
                            1 if dtype == "bf16" else 0)
        self._refresh()

    def _refresh(self):
        self._ca = _Cache(*[_p(a) for a in (self.k_cache, self.v_cache, self.codes, self.scores, self.pos,
                                            self.budget, self.fill, self.next_pos)])

    def reset(self):
        _load().orc_reset(ctypes.byref(self._cfg), ctypes.byref(self._ca))

    def step(self, W, q, k, v):
        """Algorithm 1 lines 1-5 from embeddings. q [B, H*G, d], k / v [B, H, d]. Returns victim, evicted_pos, qcodes, kcodes."""
        B, H, G, Wd = self.B, self.H, self.G, self.Wd
        victim = np.zeros((B, H), dtype=np.int32)
        evicted = np.zeros((B, H), dtype=np.int32)
        qcodes = np.zeros((B, H * G, Wd), dtype=np.uint32)
        kcodes = np.zeros((B, H, Wd), dtype=np.uint32)
        for a in (W, q, k, v):
            assert a.flags.c_contiguous
        _load().orc_step(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(W), _p(q), _p(k), _p(v), _p(victim), _p(evicted),
                         _p(qcodes), _p(kcodes), self.threads)
        return victim, evicted, qcodes, kcodes

    def step_codes(self, qcodes, kcodes, k, v):
        """Algorithm 1 lines 1-5 on given codes (qcodes [B, H*G, Wd], kcodes [B, H, Wd])."""
        victim = np.zeros((self.B, self.H), dtype=np.int32)
        evicted = np.zeros((self.B, self.H), dtype=np.int32)
        qcodes = np.ascontiguousarray(qcodes, dtype=np.uint32)
        kcodes = np.ascontiguousarray(kcodes, dtype=np.uint32)
        assert k.flags.c_contiguous and v.flags.c_contiguous
        _load().orc_step_codes(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(qcodes), _p(kcodes), _p(k), _p(v),
                               _p(victim), _p(evicted), self.threads)
        return victim, evicted

    def oneshot_codes(self, kcodes, qcodes, k, v, prompt_len, want_sums=False):
        """One-shot ranking by averaged Hamming distance (Appendix C) on given codes; fills the cache with the kept tokens."""
        Nmax = k.shape[2]
        plen = np.ascontiguousarray(prompt_len, dtype=np.int32)
        kcodes = np.ascontiguousarray(kcodes, dtype=np.uint32)
        qcodes = np.ascontiguousarray(qcodes, dtype=np.uint32)
        assert kcodes.shape == (self.B, self.H, Nmax, self.Wd) and qcodes.shape == (self.B, self.H, Nmax, self.G, self.Wd)
        assert k.strides == v.strides
        ks = self._strides(k)
        sums = np.zeros((self.B, self.H, Nmax), dtype=np.int64) if want_sums else None
        _load().orc_oneshot_codes(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(kcodes), _p(qcodes), _p(k), _p(v),
                                  _p(ks), _p(plen), Nmax, _p(sums), self.threads)
        return sums

    def oneshot_l2(self, kcodes, k, v, prompt_len, want_norms=False):
        """One-shot ranking by key L2 norm (the comparison policy the paper names); fills the cache with the kept tokens."""
        Nmax = k.shape[2]
        plen = np.ascontiguousarray(prompt_len, dtype=np.int32)
        kcodes = np.ascontiguousarray(kcodes, dtype=np.uint32)
        assert kcodes.shape == (self.B, self.H, Nmax, self.Wd) and k.strides == v.strides
        ks = self._strides(k)
        norms = np.zeros((self.B, self.H, Nmax), dtype=np.float32) if want_norms else None
        _load().orc_oneshot_l2(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(kcodes), _p(k), _p(v), _p(ks), _p(plen), Nmax,
                               _p(norms), self.threads)
        return norms

    def step_l2(self, k, v):
        """One decoding step of the L2-norm comparison policy. k / v [B, H, d]. Returns victim, evicted_pos."""
        victim = np.zeros((self.B, self.H), dtype=np.int32)
        evicted = np.zeros((self.B, self.H), dtype=np.int32)
        assert k.flags.c_contiguous and v.flags.c_contiguous
        _load().orc_step_l2(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(k), _p(v), _p(victim), _p(evicted), self.threads)
        return victim, evicted

    def attention_loss(self, q, k_full):
        """1 - attention mass of the cached tokens under q over all next_pos tokens seen. q [B, H*G, d] -> fp64 [B, H*G]."""
        assert q.flags.c_contiguous and q.shape == (self.B, self.H * self.G, self.d)
        ks = self._strides(k_full)
        out = np.zeros((self.B, self.H * self.G), dtype=np.float64)
        _load().orc_attention_loss(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(q), _p(k_full), _p(ks), _p(out))
        return out

    def attend(self, q):
        """Eq. 1 over the compressed cache (Algorithm 1 line 6). q [B, H*G, d] -> fp64 [B, H*G, d]."""
        assert q.flags.c_contiguous and q.shape == (self.B, self.H * self.G, self.d)
        out = np.zeros((self.B, self.H * self.G, self.d), dtype=np.float64)
        _load().orc_attend(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(q), _p(out))
        return out

    @staticmethod
    def _strides(a):
        es = a.itemsize
        assert a.strides[3] == es
        return np.array([a.strides[0] // es, a.strides[1] // es, a.strides[2] // es], dtype=np.int64)

    def prefill(self, W, q, k, v, prompt_len, want_codes=False):
        """Prompt Encoding Stage from embeddings. q [B, H*G, Nmax, d], k / v [B, H, Nmax, d] (any strides on the first three axes)."""
        Nmax = k.shape[2]
        plen = np.ascontiguousarray(prompt_len, dtype=np.int32)
        assert k.strides == v.strides
        qs, ks = self._strides(q), self._strides(k)
        kc = np.zeros((self.B, self.H, Nmax, self.Wd), dtype=np.uint32) if want_codes else None
        qc = np.zeros((self.B, self.H, Nmax, self.G, self.Wd), dtype=np.uint32) if want_codes else None
        _load().orc_prefill(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(W), _p(q), _p(k), _p(v), _p(qs), _p(ks),
                            _p(plen), Nmax, _p(kc), _p(qc), self.threads)
        return (kc, qc) if want_codes else None

    def prefill_codes(self, kcodes, qcodes, k, v, prompt_len):
        """Prompt Encoding Stage on given codes (kcodes [B, H, Nmax, Wd], qcodes [B, H, Nmax, G, Wd])."""
        Nmax = k.shape[2]
        plen = np.ascontiguousarray(prompt_len, dtype=np.int32)
        kcodes = np.ascontiguousarray(kcodes, dtype=np.uint32)
        qcodes = np.ascontiguousarray(qcodes, dtype=np.uint32)
        assert kcodes.shape == (self.B, self.H, Nmax, self.Wd) and qcodes.shape == (self.B, self.H, Nmax, self.G, self.Wd)
        assert k.strides == v.strides
        ks = self._strides(k)
        _load().orc_prefill_codes(ctypes.byref(self._cfg), ctypes.byref(self._ca), _p(kcodes), _p(qcodes), _p(k), _p(v),
                                  _p(ks), _p(plen), Nmax, self.threads)
