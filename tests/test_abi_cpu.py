"""CPU-only checks of the C ABI: the library loads, exports every declared symbol, and the
host-side validation returns the documented status codes without touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build_mod.build()
    return B.lib()


def test_every_declared_symbol_is_exported(L):
    declared = set()
    for name in sorted(os.listdir(os.path.join(ROOT, "include"))):
        hdr = open(os.path.join(ROOT, "include", name)).read()
        hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
        declared |= set(re.findall(r"\b(okq_[a-z_]+)\s*\(", hdr))
    assert declared == set(B.exported_symbols())
    for s in declared:
        assert hasattr(L, s), s


def test_status_strings(L):
    assert L.okq_status_string(0) == b"ok"
    assert L.okq_status_string(B.ERR_TIMEOUT) == b"bounded device wait timed out"   # the device status of a wait that ran out
    seen = {L.okq_status_string(i) for i in range(8)}
    assert len(seen) == 8
    assert L.okq_last_cuda_error() == 0


def test_cache_sizes_and_record_format(L):
    s = B.cache_sizes(28, 8, 4, 28, 16384)
    units = 28 * 8 * 4
    assert s[0] == units * (16384 // 32) * 2688
    # 2688 B per 32-token window = 84 B per token per KV head = 2.625 bits per element
    assert B.RECORD_BYTES / 32 == 84 and B.RECORD_BYTES * 8 / (32 * 2 * 128) == 2.625
    assert s[1] == 8 * 16384 and s[2] == s[3] == units * 32 * 128 * 2 and s[4] == 28 * 8 * 4


def test_shape_validation(L):
    def sizes(**kw):
        d = dict(n_layers=1, batch=1, n_kv_heads=1, n_q_heads=7, head_dim=128, window=32, capacity=64)
        d.update(kw)
        c = B.okq_cache(d["n_layers"], d["batch"], d["n_kv_heads"], d["n_q_heads"], d["head_dim"], d["window"],
                        d["capacity"], 0, 0, 0)
        out = (C.c_size_t * 6)()
        return L.okq_cache_sizes(C.byref(c), out)
    assert sizes() == B.OK
    assert sizes(head_dim=64) == B.ERR_UNSUPPORTED
    assert sizes(window=16) == B.ERR_UNSUPPORTED
    assert sizes(n_q_heads=9) == B.ERR_UNSUPPORTED          # group 9 > 8
    assert sizes(n_kv_heads=2, n_q_heads=7) == B.ERR_UNSUPPORTED
    assert sizes(capacity=70) == B.ERR_INVALID_ARG
    assert sizes(batch=0) == B.ERR_INVALID_ARG


def test_pointer_validation_before_any_launch(L):
    c = B.okq_cache(1, 1, 1, 7, 128, 32, 64, 0, 0, 0, 0, 0, 0, 0, 0, 0)
    strides = (C.c_int64 * 3)(64 * 128, 64 * 128, 128)
    assert L.okq_quantize_keys(C.byref(c), 0, 4096, strides, 64, 4096, None) == B.ERR_INVALID_ARG   # null buffers
    fake = 1 << 20
    c = B.okq_cache(1, 1, 1, 7, 128, 32, 64, 0, 0, 0, fake, fake, fake, fake, fake, fake)
    assert L.okq_quantize_keys(C.byref(c), 1, fake, strides, 64, fake, None) == B.ERR_INVALID_ARG   # layer out of range
    assert L.okq_quantize_keys(C.byref(c), 0, fake, strides, 96, fake, None) == B.ERR_CAPACITY
    assert L.okq_quantize_keys(C.byref(c), 0, fake + 2, strides, 64, fake, None) == B.ERR_ALIGNMENT
    bad = (C.c_int64 * 3)(64 * 128, 64 * 128, 100)
    assert L.okq_quantize_keys(C.byref(c), 0, fake, bad, 64, fake, None) == B.ERR_ALIGNMENT
    assert L.okq_quantize_values(C.byref(c), 0, fake, strides, 64, fake, fake, 2, None) == B.ERR_INVALID_ARG  # n_R
    assert L.okq_append(C.byref(c), 0, 2, fake, fake, fake, fake, fake, 1, None) == B.ERR_INVALID_ARG
    assert L.okq_decode_attention(C.byref(c), 0, 1, fake, 0.1, fake, fake, 1, fake, 16, 0, fake, None) == B.ERR_WORKSPACE
    assert L.okq_decode_workspace_bytes(C.byref(c), 1, 3) > 0
    assert L.okq_decode_workspace_bytes(C.byref(c), 0, 3) == 0
    c8 = B.okq_cache(1, 1, 1, 7, 128, 32, 64, 0, 0, 0, fake + 8, fake, fake, fake, fake, fake)
    assert L.okq_append(C.byref(c8), 0, 1, fake, fake, fake, fake, fake, 1, None) == B.ERR_ALIGNMENT


def test_calibration_argument_checks(L):
    assert L.okq_calib_workspace_bytes(0, 16) == 0 and L.okq_calib_workspace_bytes(7, 0) == 0
    # the largest of: row statistics + per-(query tile, head) column sums; 64 partial moment sets; 128 x 128 fp64
    assert L.okq_calib_workspace_bytes(7, 4096) >= max((7 * 4096 * 2 + 64 * 7 * 4096) * 4, 64 * 3 * 128 * 128 * 4, 128 * 128 * 8)
    assert L.okq_calib_workspace_bytes(1, 8) >= 64 * 3 * 128 * 128 * 4
    null = C.c_void_p(0)
    assert L.okq_calib_attention_weights(null, null, 7, 64, C.c_float(1.0), 1, null, 0, null, null) == B.ERR_INVALID_ARG
    assert L.okq_calib_moments(null, null, null, 64, null, 0, null, null) == B.ERR_INVALID_ARG
    assert L.okq_calib_rotation(null, null, null, 0, null, null, null, null) == B.ERR_INVALID_ARG
    fake = C.c_void_p(4096)      # aligned, never dereferenced: the size checks come first
    assert L.okq_calib_attention_weights(fake, fake, 7, 64, C.c_float(1.0), 1, fake, 16, fake, null) == B.ERR_WORKSPACE
    assert L.okq_calib_attention_weights(C.c_void_p(4100), fake, 7, 64, C.c_float(1.0), 1, fake, 1 << 30, fake, null) == B.ERR_ALIGNMENT
    assert L.okq_calib_rotation(fake, fake, fake, 1024, fake, fake, null, null) == B.ERR_WORKSPACE


def test_ladder_codebook_constants_equal_the_oracle_quantiser(L):
    """The value levels and thresholds compiled into the ladder kernels are the fp32 roundings of the Lloyd-Max
    quantiser of N(0, 1/128) that the oracle derives by iteration (Eq. 3)."""
    import numpy as np
    from oracle import okq_ladder_oracle as LO
    for bits in (2, 3, 4):
        lv, th = B.ladder_codebook(bits)
        olv, oth = LO.codebook32(bits)
        assert np.array_equal(np.array(lv, dtype=np.float32), olv), bits
        assert np.array_equal(np.array(th, dtype=np.float32), oth), bits
    lv, th = (C.c_float * 16)(), (C.c_float * 15)()
    assert L.okq_ladder_codebook(5, lv, th) == 0 and L.okq_ladder_codebook(1, lv, th) == 0


def test_ladder_validation_before_any_launch(L):
    fake = 1 << 20
    strides = (C.c_int64 * 3)(64 * 128, 64 * 128, 128)

    def cache(bits=3, capacity=64, n_q=7, **kw):
        ptrs = dict(k_codes=fake, k_norm=fake, k_meta=fake, v_codes=fake, v_norm=fake, modality=fake)
        ptrs.update(kw)
        return B.okq_ladder_cache(1, 1, n_q, capacity, bits, 0, ptrs["k_codes"], ptrs["k_norm"], ptrs["k_meta"],
                                  ptrs["v_codes"], ptrs["v_norm"], ptrs["modality"])
    keys = lambda c, n=64, k=fake: L.okq_ladder_quantize_keys(C.byref(c), k, strides, n, fake, None)
    assert keys(cache(bits=5)) == B.ERR_UNSUPPORTED
    assert keys(cache(bits=1)) == B.ERR_UNSUPPORTED
    assert keys(cache(n_q=9)) == B.ERR_UNSUPPORTED
    assert keys(cache(capacity=70)) == B.ERR_INVALID_ARG
    assert keys(cache(), n=48) == B.ERR_INVALID_ARG            # not a whole number of windows
    assert keys(cache(), n=96) == B.ERR_INVALID_ARG            # beyond the capacity
    assert keys(cache(k_meta=0)) == B.ERR_INVALID_ARG
    assert keys(cache(k_codes=fake + 4)) == B.ERR_ALIGNMENT
    assert keys(cache(), k=fake + 2) == B.ERR_ALIGNMENT
    assert keys(cache(), n=0) == B.OK                          # nothing to do, nothing launched
    assert L.okq_ladder_quantize_values(C.byref(cache()), fake, strides, 64, fake, fake, 2, None) == B.ERR_INVALID_ARG
    assert L.okq_ladder_decode_attention(C.byref(cache()), 64, fake, 0.1, fake, fake, 1, 0, None) == B.ERR_INVALID_ARG
