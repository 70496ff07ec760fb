"""The C ABI library builds, loads without a GPU, and exports every symbol include/hashevict.h declares."""
import ctypes
import os
import re

from paper_2412_16187_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hashevict.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(he_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert {"he_hash_keys", "he_prefill_compress", "he_decode_step", "he_reset"} <= set(names)
    L = ctypes.CDLL(build.build_cuda())
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(binding.EXPORTS)


def test_host_side_validation_needs_no_gpu():
    L = binding.lib()
    cfg = binding.he_config(2, 2, 4, 128, 64, 4096, 0, 0, 1, 1)
    assert L.he_workspace_bytes(ctypes.byref(cfg), 8192) >= 2 * 2 * 8192 * 5 * 2 * 4
    bad = binding.he_config(2, 2, 4, 128, 65, 4096, 0, 0, 1, 1)
    assert L.he_workspace_bytes(ctypes.byref(bad), 8192) == 0
    assert L.he_hash_keys(ctypes.byref(bad), None, 1, 128, None, None, None) == 1
    assert b"hash_bits" in L.he_last_error()
    odd = binding.he_config(2, 2, 4, 128, 64, 4098, 0, 0, 1, 1)
    ca = binding.he_cache()
    assert L.he_reset(ctypes.byref(odd), ctypes.byref(ca), None) == 1 and b"max_budget" in L.he_last_error()
    assert L.he_reset(ctypes.byref(cfg), ctypes.byref(ca), None) == 1 and b"null" in L.he_last_error()


def test_flag_values_match_the_header_and_packed_layout_is_validated_on_the_host():
    text = open(os.path.join(ROOT, "include", "hashevict.h")).read()
    flags = {m.group(1): int(m.group(2)) for m in re.finditer(r"#define\s+(HE_FLAG_[A-Z_]+)\s+(\d+)u", text)}
    assert flags == {"HE_FLAG_WRITE_SCORES": binding.HE_FLAG_WRITE_SCORES, "HE_FLAG_PACKED_CODES": binding.HE_FLAG_PACKED_CODES,
                     "HE_FLAG_EARLY_INPUTS": binding.HE_FLAG_EARLY_INPUTS}
    L = binding.lib()
    packed = binding.HE_FLAG_PACKED_CODES
    ca = binding.he_cache()
    # 40-bit codes would need 5 bytes per slot: only 1 to 3 bytes, or whole words, are stored
    wide = binding.he_config(1, 1, 1, 128, 40, 64, 0, 0, 1, packed)
    assert L.he_reset(ctypes.byref(wide), ctypes.byref(ca), None) == 2 and b"packed codes" in L.he_last_error()
    # one byte per slot: the slot stride must keep units 16-byte aligned
    ragged = binding.he_config(1, 1, 1, 128, 8, 36, 0, 0, 1, packed)
    assert L.he_reset(ctypes.byref(ragged), ctypes.byref(ca), None) == 1 and b"multiple of 16" in L.he_last_error()
    # 32- and 64-bit codes are the same bytes in both layouts: the flag changes nothing, the null cache is what fails
    same = binding.he_config(1, 1, 1, 128, 64, 36, 0, 0, 1, packed)
    assert L.he_reset(ctypes.byref(same), ctypes.byref(ca), None) == 1 and b"null" in L.he_last_error()


def test_budgets_outside_the_cache_are_rejected_on_the_host_when_a_mirror_is_given():
    """Budgets must lie in [1, max_budget]; with he_cache.budget_host the call fails before anything is launched
    (the pointers below are never dereferenced: the check comes first)."""
    L = binding.lib()
    cfg = binding.he_config(2, 2, 4, 128, 64, 64, 0, 0, 1, 1)
    fake = 0x10000
    for bad, word in (([0, 8], b"budget 0"), ([8, -3], b"budget -3"), ([8, 65], b"budget 65")):
        mirror = (ctypes.c_int32 * 2)(*bad)
        ca = binding.he_cache(*([fake] * 9), ctypes.cast(mirror, ctypes.c_void_p), None)
        rc = L.he_decode_step(ctypes.byref(cfg), ctypes.byref(ca), fake, fake, fake, fake, None, None, None)
        assert rc == 1 and word in L.he_last_error(), L.he_last_error()
        i64x3 = ctypes.c_int64 * 3
        rc = L.he_prefill_compress(ctypes.byref(cfg), ctypes.byref(ca), fake, fake, fake, i64x3(128, 128, 128), i64x3(128, 128, 128),
                                   fake, 16, 0x20000, 1 << 30, None)
        assert rc == 1 and word in L.he_last_error(), L.he_last_error()
