"""Python binding of the C ABI in include/hashevict.h. Argument marshalling only: every step runs in the CUDA kernels.

PyTorch provides device memory and streams. There is no CPU fallback: if the CUDA library cannot be
loaded, or a call fails, HashEvictError is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

HE_OK = 0
HE_DTYPE_F32, HE_DTYPE_BF16 = 0, 1
HE_FLAG_WRITE_SCORES = 1
HE_FLAG_PACKED_CODES = 2
HE_FLAG_EARLY_INPUTS = 4
_DTYPES = {torch.float32: HE_DTYPE_F32, torch.bfloat16: HE_DTYPE_BF16}


class HashEvictError(RuntimeError):
    pass


class he_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("batch", "n_kv_heads", "group_size", "head_dim", "hash_bits", "max_budget", "n_sink", "n_recent", "dtype")] + \
               [("flags", ctypes.c_uint32)]


class he_cache(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("k_cache", "v_cache", "codes", "scores", "pos", "budget", "fill", "next_pos", "W", "budget_host", "step_scratch")]


EXPORTS = (
    "he_hash_keys", "he_decode_step", "he_prefill_compress", "he_workspace_bytes", "he_reset",
    "he_decode_staging_bytes", "he_decode_step_host", "he_decode_step_host_enqueue", "he_decode_step_host_block_enqueue", "he_decode_host_block_bytes", "he_prefill_staging_bytes", "he_prefill_compress_host",
    "he_prefill_compress_noalloc", "he_attend", "he_prefill_oneshot", "he_oneshot_workspace_bytes", "he_prefill_oneshot_l2", "he_attention_loss", "he_decode_step_l2", "he_step_scratch_bytes", "he_device_error_count", "he_prefill_phase_events", "he_last_error",
)

_lib = None


def lib():
    """Load (building if needed) libhashevict.so and declare the signatures of include/hashevict.h."""
    global _lib
    if _lib is not None:
        return _lib
    if os.environ.get("HE_DEBUG_LIB") == "1":  # the bounds-checking build (see build.build_cuda)
        path = _build.build_cuda(debug=True)
    else:
        path = _build.build_cuda() if not os.path.exists(_build.LIB_PATH) else _build.LIB_PATH
    try:
        L = ctypes.CDLL(path)
    except OSError as e:  # no silent fallback
        raise HashEvictError(f"cannot load the CUDA library {path}: {e}") from e
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    cfgp, cap = ctypes.POINTER(he_config), ctypes.POINTER(he_cache)
    L.he_hash_keys.argtypes = [cfgp, vp, i64, i64, vp, vp, vp]
    L.he_decode_step.argtypes = [cfgp, cap, vp, vp, vp, vp, vp, vp, vp]
    L.he_prefill_compress.argtypes = [cfgp, cap, vp, vp, vp, ctypes.POINTER(i64), ctypes.POINTER(i64), vp, i32, vp, sz, vp]
    L.he_workspace_bytes.argtypes = [cfgp, i32]
    L.he_workspace_bytes.restype = sz
    L.he_reset.argtypes = [cfgp, cap, vp]
    L.he_decode_staging_bytes.argtypes = [cfgp]
    L.he_decode_staging_bytes.restype = sz
    L.he_decode_step_host.argtypes = [cfgp, cap, vp, vp, vp, vp, vp, sz, vp]
    L.he_decode_step_host_enqueue.argtypes = [cfgp, cap, vp, vp, vp, vp, vp, sz, vp]
    L.he_decode_step_host_block_enqueue.argtypes = [cfgp, cap, vp, vp, vp, sz, vp]
    L.he_decode_step_host_block_enqueue.restype = ctypes.c_int
    L.he_decode_host_block_bytes.argtypes = [cfgp, ctypes.POINTER(sz)]
    L.he_decode_host_block_bytes.restype = sz
    L.he_prefill_staging_bytes.argtypes = [cfgp, i32]
    L.he_prefill_staging_bytes.restype = sz
    L.he_prefill_compress_host.argtypes = [cfgp, cap, vp, vp, vp, vp, i32, vp, vp, sz, vp]
    L.he_prefill_compress_noalloc.argtypes = [cfgp, cap, vp, vp, vp, ctypes.POINTER(i64), ctypes.POINTER(i64), vp, i32, vp]
    L.he_prefill_oneshot.argtypes = [cfgp, cap, vp, vp, vp, ctypes.POINTER(i64), ctypes.POINTER(i64), vp, i32, vp, sz, vp, vp]
    L.he_prefill_oneshot_l2.argtypes = [cfgp, cap, vp, vp, ctypes.POINTER(i64), vp, i32, vp, sz, vp, vp]
    L.he_attention_loss.argtypes = [cfgp, cap, vp, vp, ctypes.POINTER(i64), i32, vp, vp]
    L.he_decode_step_l2.argtypes = [cfgp, cap, vp, vp, vp, vp, vp]
    L.he_oneshot_workspace_bytes.argtypes = [cfgp, i32]
    L.he_oneshot_workspace_bytes.restype = sz
    L.he_attend.argtypes = [cfgp, cap, vp, vp, vp]
    L.he_attend.restype = ctypes.c_int
    L.he_step_scratch_bytes.argtypes = [cfgp]
    L.he_step_scratch_bytes.restype = sz
    L.he_prefill_phase_events.argtypes = [ctypes.POINTER(vp)]
    L.he_prefill_phase_events.restype = ctypes.c_int
    L.he_device_error_count.argtypes = []
    L.he_device_error_count.restype = ctypes.c_int
    L.he_last_error.argtypes = []
    L.he_last_error.restype = ctypes.c_char_p
    for name in ("he_hash_keys", "he_decode_step", "he_prefill_compress", "he_reset", "he_decode_step_host", "he_decode_step_host_enqueue",
                 "he_prefill_compress_host", "he_prefill_compress_noalloc"):
        getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def device_error_count() -> int:
    """he_device_error_count: thread blocks that gave up on a bounded wait (0 in a healthy process). Synchronises."""
    return lib().he_device_error_count()


def prefill_phase_events(events=None):
    """he_prefill_phase_events: five torch.cuda.Event(enable_timing=True) that the next prefill calls of this thread
    record around their phases (hash K, hash Q, schedule + replay, gather), or None to switch that off."""
    if events is None:
        lib().he_prefill_phase_events(None)
        return
    assert len(events) == 5
    for e in events:
        e.record()  # torch creates the underlying cudaEvent lazily, on first record
    arr = (ctypes.c_void_p * 5)(*[e.cuda_event for e in events])
    lib().he_prefill_phase_events(arr)


def _check(rc: int):
    if rc != HE_OK:
        raise HashEvictError(f"hashevict error {rc}: {lib().he_last_error().decode()}")


def _stream(stream=None) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def hash_keys(x: torch.Tensor, W: torch.Tensor, hash_bits: int | None = None, stream=None) -> torch.Tensor:
    """he_hash_keys: SimHash codes [rows, Wd] (int32 bit patterns) of the rows of x [rows, d] (Eq. 2)."""
    assert x.is_cuda and W.is_cuda and x.dim() == 2 and x.stride(1) == 1 and W.dtype == torch.float32 and W.is_contiguous()
    b = W.shape[1] if hash_bits is None else hash_bits
    cfg = he_config(1, 1, 1, x.shape[1], b, 4, 0, 0, _DTYPES[x.dtype], 0)
    out = torch.empty((x.shape[0], (b + 31) // 32), dtype=torch.int32, device=x.device)
    _check(lib().he_hash_keys(ctypes.byref(cfg), _ptr(x), x.shape[0], x.stride(0), _ptr(W), _ptr(out), _stream(stream)))
    return out


def _config(batch, n_kv_heads, group_size, head_dim, hash_bits, max_budget, n_sink, n_recent, dtype, flags):
    return he_config(batch, n_kv_heads, group_size, head_dim, hash_bits, max_budget, n_sink, n_recent, _DTYPES[dtype], flags)


def workspace_bytes(cfg: he_config, max_prompt_len: int) -> int:
    return lib().he_workspace_bytes(ctypes.byref(cfg), max_prompt_len)


def decode_staging_bytes(cfg: he_config) -> int:
    return lib().he_decode_staging_bytes(ctypes.byref(cfg))


def prefill_staging_bytes(cfg: he_config, max_prompt_len: int) -> int:
    return lib().he_prefill_staging_bytes(ctypes.byref(cfg), max_prompt_len)


class HashEvictCache:
    """Device-side cache state (the arrays of he_cache, allocated with torch) plus the calls that act on it."""

    def __init__(self, batch, n_kv_heads, group_size, head_dim, hash_bits, budgets, W, dtype=torch.bfloat16,
                 max_budget=None, n_sink=0, n_recent=0, write_scores=True, device="cuda", host_budget_mirror=True,
                 packed_codes=False, early_inputs=False):
        lib()
        dev = torch.device(device)
        budgets = torch.as_tensor(budgets, dtype=torch.int32).reshape(-1)
        assert budgets.numel() == batch
        cmax = int(budgets.max()) if max_budget is None else int(max_budget)
        cmax = (cmax + 3) // 4 * 4  # the slot stride must keep 16-byte alignment
        if packed_codes:
            cmax = (cmax + 15) // 16 * 16  # ... also with one byte per slot
        self.B, self.H, self.G, self.d, self.b, self.Cmax = batch, n_kv_heads, group_size, head_dim, hash_bits, cmax
        self.Wd = (hash_bits + 31) // 32
        self.dtype = dtype
        self.k_cache = torch.zeros((batch, n_kv_heads, cmax, head_dim), dtype=dtype, device=dev)
        self.v_cache = torch.zeros_like(self.k_cache)
        # code table: Wd 32-bit words per slot, or ceil(b/8) bytes per slot with HE_FLAG_PACKED_CODES
        self.packed_codes = bool(packed_codes)
        if self.packed_codes:
            self.codes_storage = torch.zeros((batch, n_kv_heads, cmax, (hash_bits + 7) // 8), dtype=torch.uint8, device=dev)
        else:
            self.codes_storage = torch.zeros((batch, n_kv_heads, cmax, self.Wd), dtype=torch.int32, device=dev)
        self.scores = torch.zeros((batch, n_kv_heads, cmax), dtype=torch.float32, device=dev)
        self.pos = torch.full((batch, n_kv_heads, cmax), -1, dtype=torch.int32, device=dev)
        self.budget = budgets.to(dev)
        self.fill = torch.zeros((batch, n_kv_heads), dtype=torch.int32, device=dev)
        self.next_pos = torch.zeros((batch, n_kv_heads), dtype=torch.int32, device=dev)
        self.W = W.to(device=dev, dtype=torch.float32).contiguous()
        assert self.W.shape == (head_dim, hash_bits)
        self.cfg = _config(batch, n_kv_heads, group_size, head_dim, hash_bits, cmax, n_sink, n_recent, dtype,
                           (HE_FLAG_WRITE_SCORES if write_scores else 0) | (HE_FLAG_PACKED_CODES if packed_codes else 0) |
                           (HE_FLAG_EARLY_INPUTS if early_inputs else 0))
        self._budget_host = (ctypes.c_int32 * batch)(*[int(x) for x in budgets.tolist()])  # host mirror of `budget`
        self.ca = he_cache(*[_ptr(t) for t in (self.k_cache, self.v_cache, self.codes_storage, self.scores, self.pos,
                                               self.budget, self.fill, self.next_pos, self.W)],
                           ctypes.cast(self._budget_host, ctypes.c_void_p) if host_budget_mirror else None, None)
        # scratch for the bulk-hashed decode step that large batches use (codes of the step's new rows)
        self.step_scratch = torch.empty(lib().he_step_scratch_bytes(ctypes.byref(self.cfg)), dtype=torch.uint8, device=dev)
        self.ca.step_scratch = _ptr(self.step_scratch)
        self._ws = None

    @property
    def codes(self):
        """The code table as int32 words [B, Hkv, Cmax, Wd]: the storage itself, or (packed layout) a copy widened to words."""
        if not self.packed_codes:
            return self.codes_storage
        raw = self.codes_storage
        wide = torch.zeros(raw.shape[:-1] + (4 * self.Wd,), dtype=torch.uint8, device=raw.device)
        wide[..., :raw.shape[-1]] = raw
        return wide.view(torch.int32)

    # --- the four calls of the boundary -------------------------------------------------------------
    def reset(self, stream=None):
        _check(lib().he_reset(ctypes.byref(self.cfg), ctypes.byref(self.ca), _stream(stream)))

    def decode_step(self, q, k, v, victim_out=None, evicted_pos_out=None, qcodes_out=None, stream=None):
        """he_decode_step. q [B, H*G, d], k / v [B, H, d], contiguous. Returns victim_out [B, H] (int32)."""
        if victim_out is None:
            victim_out = torch.empty((self.B, self.H), dtype=torch.int32, device=self.k_cache.device)
        _check(lib().he_decode_step(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q), _ptr(k), _ptr(v),
                                    _ptr(victim_out), _ptr(evicted_pos_out), _ptr(qcodes_out), _stream(stream)))
        return victim_out

    def attend(self, q, out=None, stream=None):
        """he_attend: softmax(q K^T / sqrt(d)) V over the valid slots (Eq. 1). q [B, H*G, d] -> fp32 [B, H*G, d]."""
        if out is None:
            out = torch.empty((self.B, self.H * self.G, self.d), dtype=torch.float32, device=self.k_cache.device)
        _check(lib().he_attend(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q), _ptr(out), _stream(stream)))
        return out

    def workspace(self, max_prompt_len):
        need = workspace_bytes(self.cfg, max_prompt_len)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.k_cache.device)
        return self._ws

    def prefill_compress(self, q, k, v, prompt_len, max_prompt_len=None, workspace=None, stream=None):
        """he_prefill_compress. q [B, H*G, N, d], k / v [B, H, N, d] (any strides on the first three axes);
        prompt_len int32 [B] on the device."""
        nmax = k.shape[2] if max_prompt_len is None else max_prompt_len
        ws = self.workspace(nmax) if workspace is None else workspace
        assert q.stride(3) == 1 and k.stride(3) == 1 and k.stride() == v.stride()
        i64x3 = ctypes.c_int64 * 3
        _check(lib().he_prefill_compress(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q), _ptr(k), _ptr(v),
                                         i64x3(*q.stride()[:3]), i64x3(*k.stride()[:3]), _ptr(prompt_len), nmax,
                                         _ptr(ws), ws.numel(), _stream(stream)))

    def prefill_oneshot(self, q, k, v, prompt_len, max_prompt_len=None, sums_out=None, stream=None):
        """he_prefill_oneshot: the averaged-Hamming ranking of Appendix C instead of Algorithm 1 (same arguments as
        prefill_compress; sums_out int64 [B, H, Nmax] optionally receives the summed distances)."""
        nmax = k.shape[2] if max_prompt_len is None else max_prompt_len
        need = lib().he_oneshot_workspace_bytes(ctypes.byref(self.cfg), nmax)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.k_cache.device)
        assert q.stride(3) == 1 and k.stride(3) == 1 and k.stride() == v.stride()
        i64x3 = ctypes.c_int64 * 3
        _check(lib().he_prefill_oneshot(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q), _ptr(k), _ptr(v),
                                        i64x3(*q.stride()[:3]), i64x3(*k.stride()[:3]), _ptr(prompt_len), nmax,
                                        _ptr(self._ws), self._ws.numel(), _ptr(sums_out), _stream(stream)))

    def prefill_oneshot_l2(self, k, v, prompt_len, max_prompt_len=None, norms_out=None, stream=None):
        """he_prefill_oneshot_l2: keep the min(N, C) prompt tokens with the lowest key L2 norm (the comparison policy)."""
        nmax = k.shape[2] if max_prompt_len is None else max_prompt_len
        need = lib().he_oneshot_workspace_bytes(ctypes.byref(self.cfg), nmax)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.k_cache.device)
        assert k.stride(3) == 1 and k.stride() == v.stride()
        i64x3 = ctypes.c_int64 * 3
        _check(lib().he_prefill_oneshot_l2(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(k), _ptr(v), i64x3(*k.stride()[:3]),
                                           _ptr(prompt_len), nmax, _ptr(self._ws), self._ws.numel(), _ptr(norms_out), _stream(stream)))

    def decode_step_l2(self, k, v, victim_out=None, evicted_pos_out=None, stream=None):
        """he_decode_step_l2: one step of the L2-norm comparison policy. k / v [B, H, d]. Returns victim_out [B, H]."""
        if victim_out is None:
            victim_out = torch.empty((self.B, self.H), dtype=torch.int32, device=self.k_cache.device)
        _check(lib().he_decode_step_l2(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(k), _ptr(v), _ptr(victim_out),
                                       _ptr(evicted_pos_out), _stream(stream)))
        return victim_out

    def attention_loss(self, q, k_full, out=None, stream=None):
        """he_attention_loss: attention mass of the tokens that are no longer cached. q [B, H*G, d], k_full [B, H, n, d] -> fp32 [B, H*G]."""
        if out is None:
            out = torch.empty((self.B, self.H * self.G), dtype=torch.float32, device=self.k_cache.device)
        assert k_full.stride(3) == 1
        i64x3 = ctypes.c_int64 * 3
        _check(lib().he_attention_loss(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q), _ptr(k_full), i64x3(*k_full.stride()[:3]),
                                       k_full.shape[2], _ptr(out), _stream(stream)))
        return out

    def prefill_compress_noalloc(self, q, k, v, prompt_len, max_prompt_len=None, stream=None):
        """he_prefill_compress_noalloc: same call, prompt codes go to the library's built-in scratch (no workspace,
        no allocation). Raises HashEvictError when the prompt codes would not fit HE_NOALLOC_SCRATCH_BYTES."""
        nmax = k.shape[2] if max_prompt_len is None else max_prompt_len
        assert q.stride(3) == 1 and k.stride(3) == 1 and k.stride() == v.stride()
        i64x3 = ctypes.c_int64 * 3
        _check(lib().he_prefill_compress_noalloc(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q), _ptr(k), _ptr(v),
                                                 i64x3(*q.stride()[:3]), i64x3(*k.stride()[:3]), _ptr(prompt_len), nmax,
                                                 _stream(stream)))

    def prompt_codes(self, max_prompt_len):
        """Views of the prompt codes he_prefill_compress left in the workspace: keys [B, H, Nmax, Wd], queries [B, H, Nmax, G, Wd]."""
        units = self.B * self.H
        kbytes = (units * max_prompt_len * self.Wd * 4 + 255) // 256 * 256
        ws = self._ws
        kc = ws[:units * max_prompt_len * self.Wd * 4].view(torch.int32).view(self.B, self.H, max_prompt_len, self.Wd)
        qn = units * max_prompt_len * self.G * self.Wd * 4
        qc = ws[kbytes:kbytes + qn].view(torch.int32).view(self.B, self.H, max_prompt_len, self.G, self.Wd)
        return kc, qc

    # --- host-buffer variants ------------------------------------------------------------------------
    def decode_step_host(self, q_host, k_host, v_host, victim_host, staging, stream=None):
        _check(lib().he_decode_step_host(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q_host), _ptr(k_host),
                                         _ptr(v_host), _ptr(victim_host), _ptr(staging), staging.numel(), _stream(stream)))

    def decode_step_host_enqueue(self, q_host, k_host, v_host, victim_host, staging, stream=None):
        """he_decode_step_host_enqueue: as decode_step_host but without the final synchronise (results after a stream sync)."""
        _check(lib().he_decode_step_host_enqueue(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q_host), _ptr(k_host),
                                                 _ptr(v_host), _ptr(victim_host), _ptr(staging), staging.numel(), _stream(stream)))

    def host_block_layout(self):
        """he_decode_host_block_bytes: (bytes of the one-block host layout of a step's q, k, v; their three offsets)."""
        offs = (ctypes.c_size_t * 3)()
        n = lib().he_decode_host_block_bytes(ctypes.byref(self.cfg), offs)
        return n, tuple(offs)

    def decode_step_host_block_enqueue_raw(self, qkv_ptr, victim_ptr, staging_ptr, staging_bytes, stream_ptr):
        """he_decode_step_host_block_enqueue on addresses the caller has already looked up (a serving loop reuses its
        pinned buffers, so it need not ask torch for data_ptr() and the stream handle at every step)."""
        _check(lib().he_decode_step_host_block_enqueue(ctypes.byref(self.cfg), ctypes.byref(self.ca), qkv_ptr, victim_ptr,
                                                       staging_ptr, staging_bytes, stream_ptr))

    def prefill_compress_host(self, q_host, k_host, v_host, prompt_len_host, max_prompt_len, fill_host, staging, stream=None):
        _check(lib().he_prefill_compress_host(ctypes.byref(self.cfg), ctypes.byref(self.ca), _ptr(q_host), _ptr(k_host),
                                              _ptr(v_host), _ptr(prompt_len_host), max_prompt_len, _ptr(fill_host),
                                              _ptr(staging), staging.numel(), _stream(stream)))
