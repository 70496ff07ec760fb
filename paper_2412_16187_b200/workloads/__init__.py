"""Seeded synthetic workloads shaped like the paper's runs (Section 4, "Configuration and Setup").

This module is fixture code shared by the tests and the benchmark. It holds none of the
method's arithmetic: it only produces the K / Q / V / W bytes (from the C generator in
``gen.c``) and names the five workload shapes. Both the CPU oracle and the CUDA library
consume these arrays unchanged; bf16 tensors are carried as ``uint16`` bit patterns.

Streams of the counter-based generator: 0 = W, 1/2/3 = K/Q/V noise (prompt and decode
tokens share one token axis), 7 = outlier-channel choice, 8 = drift amplitudes,
9 = cluster centres, 10 = cluster assignment, 11 = per-sequence budgets.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libhe_workloads.so")
_SRC_PATH = os.path.join(_HERE, "gen.c")
_lib = None

STREAM_W, STREAM_K, STREAM_Q, STREAM_V, STREAM_BUDGET = 0, 1, 2, 3, 11
KIND_IID, KIND_DRIFT, KIND_CLUSTER = 0, 1, 2


class _Spec(ctypes.Structure):
    _fields_ = [
        ("seed", ctypes.c_uint64),
        ("kind", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("n_heads", ctypes.c_int64),
        ("tok_space", ctypes.c_int64),
        ("d", ctypes.c_int64),
        ("noise_stream", ctypes.c_int32),
        ("n_outlier", ctypes.c_int32),
        ("outlier_scale", ctypes.c_double),
        ("drift_den", ctypes.c_double),
        ("n_clusters", ctypes.c_int32),
        ("pad_", ctypes.c_int32),
        ("centre_scale", ctypes.c_double),
        ("sigma", ctypes.c_double),
    ]


def build(force: bool = False) -> str:
    """Compile gen.c into libhe_workloads.so next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC_PATH):
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off", "-o", tmp, _SRC_PATH, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.he_gen_u64.argtypes = [ctypes.c_uint64, ctypes.c_int32, ctypes.c_uint64, ctypes.c_int64, ctypes.c_void_p]
        lib.he_gen_u64.restype = None
        lib.he_gen_normal_f32.argtypes = [ctypes.c_uint64, ctypes.c_int32, ctypes.c_uint64, ctypes.c_int64, ctypes.c_void_p]
        lib.he_gen_normal_f32.restype = None
        lib.he_gen_fill.argtypes = [ctypes.POINTER(_Spec)] + [ctypes.c_int64] * 4 + [ctypes.c_void_p] + [ctypes.c_int64] * 3
        lib.he_gen_fill.restype = None
        _lib = lib
    return _lib


@dataclass(frozen=True)
class Workload:
    """One synthetic configuration. Layers are folded into the sequence axis (n_seq = layers * batch)."""

    name: str
    seed: int
    layers: int
    batch: int
    n_kv_heads: int
    group_size: int
    head_dim: int
    dtype: str  # "f32" | "bf16"
    hash_bits: int
    prompt_len: int  # for ragged workloads: ignored, prompt = prompt_factor * budget
    budget: int  # for ragged workloads: ignored
    decode_steps: int
    key_kind: int
    ragged: bool = False
    budget_lo: int = 0
    budget_hi: int = 0
    prompt_factor: int = 2
    n_sink: int = 0
    n_recent: int = 0

    @property
    def n_seq(self) -> int:
        return self.layers * self.batch

    @property
    def n_units(self) -> int:
        return self.n_seq * self.n_kv_heads

    @property
    def words(self) -> int:
        return (self.hash_bits + 31) // 32

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    def budgets(self) -> np.ndarray:
        """Per-sequence cache budget C_s (int32[n_seq])."""
        if not self.ragged:
            return np.full(self.n_seq, self.budget, dtype=np.int32)
        raw = np.empty(self.n_seq, dtype=np.uint64)
        _load().he_gen_u64(self.seed, STREAM_BUDGET, 0, self.n_seq, raw.ctypes.data)
        span = np.uint64(self.budget_hi - self.budget_lo + 1)
        return (self.budget_lo + (raw % span).astype(np.int64)).astype(np.int32)

    def prompt_lens(self) -> np.ndarray:
        """Per-sequence prompt length N_s (int32[n_seq])."""
        if not self.ragged:
            return np.full(self.n_seq, self.prompt_len, dtype=np.int32)
        return (self.budgets().astype(np.int64) * self.prompt_factor).astype(np.int32)

    @property
    def max_budget(self) -> int:
        return int(self.budgets().max())

    @property
    def max_prompt_len(self) -> int:
        return int(self.prompt_lens().max())

    @property
    def tok_space(self) -> int:
        return self.max_prompt_len + self.decode_steps

    def scaled(self, **kw) -> "Workload":
        """A copy with some fields replaced (reduced sizes for oracle-speed parity cases)."""
        return replace(self, **kw)


# The five configurations (Section 4 shapes; budgets 10-90 % of the prompt, group size 4, Llama head_dim 128).
CONFIGS = {
    "tiny": Workload("tiny", 0, 1, 1, 4, 1, 64, "f32", 8, 128, 64, 64, KIND_IID),
    "llama2_7b_layer": Workload("llama2_7b_layer", 2, 1, 1, 32, 1, 128, "bf16", 32, 4096, 2048, 256, KIND_DRIFT),
    "llama3_8b_gqa": Workload("llama3_8b_gqa", 3, 1, 16, 8, 4, 128, "bf16", 16, 8192, 1024, 512, KIND_DRIFT),
    "long_prefill": Workload("long_prefill", 4, 32, 1, 8, 4, 128, "bf16", 32, 32768, 9830, 128, KIND_DRIFT),
    "throughput_batch": Workload(
        "throughput_batch", 5, 1, 64, 8, 4, 128, "bf16", 64, 0, 0, 1024, KIND_CLUSTER,
        ragged=True, budget_lo=512, budget_hi=4096, prompt_factor=2,
    ),
}


def _spec(w: Workload, which: str) -> _Spec:
    stream = {"k": STREAM_K, "q": STREAM_Q, "v": STREAM_V}[which]
    kind = w.key_kind if which == "k" else KIND_IID
    heads = w.n_kv_heads * (w.group_size if which == "q" else 1)
    return _Spec(
        seed=w.seed, kind=kind, dtype=1 if w.dtype == "bf16" else 0, n_heads=heads, tok_space=w.tok_space,
        d=w.head_dim, noise_stream=stream, n_outlier=4, outlier_scale=10.0, drift_den=float(w.tok_space),
        n_clusters=16, pad_=0, centre_scale=2.0, sigma=0.5,
    )


def np_dtype(w: Workload):
    return np.uint16 if w.dtype == "bf16" else np.float32


def gen_W(w: Workload, layer: int = 0) -> np.ndarray:
    """Projection matrix W[head_dim, hash_bits] = R^T, iid N(0,1) fp32 (Eq. 2's R); one per layer index."""
    n = w.head_dim * w.hash_bits
    out = np.empty(n, dtype=np.float32)
    _load().he_gen_normal_f32(w.seed, STREAM_W, layer * n, n, out.ctypes.data)
    return out.reshape(w.head_dim, w.hash_bits)


def gen_tokens(w: Workload, which: str, seq0: int, nseq: int, tok0: int, ntok: int, out: np.ndarray | None = None) -> np.ndarray:
    """Tokens [tok0, tok0+ntok) of sequences [seq0, seq0+nseq): array [nseq, heads, ntok, d] (bf16 as uint16)."""
    spec = _spec(w, which)
    heads, d = int(spec.n_heads), w.head_dim
    if out is None:
        out = np.empty((nseq, heads, ntok, d), dtype=np_dtype(w))
    assert out.shape == (nseq, heads, ntok, d) and out.flags.c_contiguous
    _load().he_gen_fill(ctypes.byref(spec), seq0, nseq, tok0, ntok, out.ctypes.data, heads * ntok * d, ntok * d, d)
    return out


def gen_decode_inputs(w: Workload, which: str, step0: int, nsteps: int) -> np.ndarray:
    """Decode-step inputs [nsteps, n_seq, heads, d]; step i of sequence s is token N_s + i of that sequence."""
    spec = _spec(w, which)
    heads, d = int(spec.n_heads), w.head_dim
    out = np.empty((nsteps, w.n_seq, heads, d), dtype=np_dtype(w))
    lens = w.prompt_lens()
    lib = _load()
    esz = out.itemsize
    if not w.ragged:
        lib.he_gen_fill(ctypes.byref(spec), 0, w.n_seq, int(lens[0]) + step0, nsteps, out.ctypes.data,
                        heads * d, d, w.n_seq * heads * d)
    else:
        for s in range(w.n_seq):
            lib.he_gen_fill(ctypes.byref(spec), s, 1, int(lens[s]) + step0, nsteps,
                            out.ctypes.data + s * heads * d * esz, heads * d, d, w.n_seq * heads * d)
    return out


def bf16_to_f32(a: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float32."""
    return (a.astype(np.uint32) << np.uint32(16)).view(np.float32)


def as_f64(w: Workload, a: np.ndarray) -> np.ndarray:
    return (bf16_to_f32(a) if w.dtype == "bf16" else a).astype(np.float64)
