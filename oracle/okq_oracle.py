"""ctypes loader for the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  The product package never does.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "okq_oracle.c")
_LIB = os.path.join(_HERE, "libokq_oracle.so")
_lib = None

D, W = 128, 32


def build(force: bool = False) -> str:
    """Compile the oracle with every fp32 operation rounded on its own (no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC",
               "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        L.okqo_half_to_float.restype = C.c_float
        L.okqo_half_to_float.argtypes = [C.c_uint16]
        L.okqo_float_to_half.restype = C.c_uint16
        L.okqo_float_to_half.argtypes = [C.c_float]
        L.okqo_bytes_per_token_head.restype = C.c_int
        L.okqo_quantize_keys.restype = C.c_int64
        L.okqo_quantize_values.restype = C.c_int64
        L.okqo_attention_batch.restype = C.c_int
        L.okqo_quantize_batch.restype = C.c_int
        L.okqo_quantize_batch_fmt.restype = C.c_int
        L.okqo_bytes_per_window_mx.restype = C.c_int
        L.okqo_mx_scale_exp.restype = C.c_int
        L.okqo_mx_scale_exp.argtypes = [C.c_float]
        L.okqo_mx_encode.restype = C.c_uint8
        L.okqo_mx_encode.argtypes = [C.c_float, C.c_int]
        L.okqo_mx_decode.restype = C.c_float
        L.okqo_mx_decode.argtypes = [C.c_uint8, C.c_int]
        _lib = L
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def half_to_float(bits: np.ndarray) -> np.ndarray:
    L = lib()
    return np.array([L.okqo_half_to_float(int(b)) for b in np.asarray(bits).ravel()], dtype=np.float32)


def float_to_half(x: np.ndarray) -> np.ndarray:
    L = lib()
    return np.array([L.okqo_float_to_half(float(v)) for v in np.asarray(x, dtype=np.float32).ravel()],
                    dtype=np.uint16)


def codebook():
    lv = (C.c_float * 4)()
    t = C.c_float()
    lib().okqo_codebook(lv, C.byref(t))
    return np.array(list(lv), dtype=np.float32), np.float32(t.value)


def bytes_per_token_head() -> int:
    return lib().okqo_bytes_per_token_head()


def fwht128(y: np.ndarray) -> np.ndarray:
    y = _c(y, np.float32).copy()
    assert y.shape == (D,)
    lib().okqo_fwht128(_p(y))
    return y


def key_rotate(k_bits: np.ndarray, signs: np.ndarray):
    """One key (uint16 fp16 bits [128]) -> (stored norm bits, z float32 [128])."""
    k_bits = _c(k_bits, np.uint16)
    signs = _c(signs, np.float32)
    z = np.empty(D, np.float32)
    n = C.c_uint16()
    lib().okqo_key_rotate(_p(k_bits), _p(signs), C.byref(n), _p(z))
    return np.uint16(n.value), z


def value_rotate(v_bits: np.ndarray, Rm: np.ndarray):
    v_bits = _c(v_bits, np.uint16)
    Rm = _c(Rm, np.float32)
    z = np.empty(D, np.float32)
    n = C.c_uint16()
    lib().okqo_value_rotate(_p(v_bits), _p(Rm), C.byref(n), _p(z))
    return np.uint16(n.value), z


def window_quantize(z: np.ndarray):
    """z float32 [32,128] -> (meta uint16 [128,2], codes uint8 [32,32])."""
    z = _c(z, np.float32)
    assert z.shape == (W, D)
    meta = np.empty((D, 2), np.uint16)
    codes = np.empty((W, D // 4), np.uint8)
    lib().okqo_window_quantize(_p(z), _p(meta), _p(codes))
    return meta, codes


def window_quantize_mx(z: np.ndarray):
    """MXFP4-metadata form of window_quantize: (mx bytes uint8 [136], decoded meta uint16 [128,2], codes [32,32])."""
    z = _c(z, np.float32)
    assert z.shape == (W, D)
    mx = np.empty(136, np.uint8)
    meta = np.empty((D, 2), np.uint16)
    codes = np.empty((W, D // 4), np.uint8)
    lib().okqo_window_quantize_mx(_p(z), _p(mx), _p(meta), _p(codes))
    return mx, meta, codes


def mx_unpack(mx: np.ndarray):
    """Stored MXFP4 bytes [..., 136] -> (m nibbles [...,128], s nibbles [...,128], m exponents [...,4], s exponents [...,4])."""
    mx = np.asarray(mx, np.uint8)
    nib = lambda b: np.stack([b & 15, b >> 4], axis=-1).reshape(*b.shape[:-1], D)
    return nib(mx[..., :64]), nib(mx[..., 64:128]), mx[..., 128:132].astype(np.int32) - 127, mx[..., 132:136].astype(np.int32) - 127


def quantize_keys(k_bits: np.ndarray, signs: np.ndarray):
    """k_bits uint16 [n,128] -> dict(codes [np,32] u8, norm [np] u16, meta [np/32,128,2] u16)."""
    k_bits = _c(k_bits, np.uint16)
    n = k_bits.shape[0]
    npk = (n // W) * W
    codes = np.zeros((npk, D // 4), np.uint8)
    norm = np.zeros(npk, np.uint16)
    meta = np.zeros((npk // W, D, 2), np.uint16)
    r = lib().okqo_quantize_keys(_p(k_bits), C.c_int64(n), _p(_c(signs, np.float32)), _p(codes), _p(norm), _p(meta))
    assert r == npk
    return {"codes": codes, "norm": norm, "meta": meta}


def quantize_values(v_bits: np.ndarray, modality: np.ndarray, R: np.ndarray):
    v_bits = _c(v_bits, np.uint16)
    n = v_bits.shape[0]
    npk = (n // W) * W
    codes = np.zeros((npk, D // 4), np.uint8)
    norm = np.zeros(npk, np.uint16)
    assert np.asarray(modality).max(initial=0) <= 2, "modality ids are 0 text, 1 audio, 2 video"
    r = lib().okqo_quantize_values(_p(v_bits), C.c_int64(n), _p(_c(modality, np.uint8)), _p(_c(R, np.float32)),
                                   _p(codes), _p(norm))
    assert r == npk
    return {"codes": codes, "norm": norm}


def dequant_key(codes, norm, meta, signs):
    out = np.empty(D, np.float64)
    lib().okqo_dequant_key(_p(_c(codes, np.uint8)), C.c_uint16(int(norm)), _p(_c(meta, np.uint16)),
                           _p(_c(signs, np.float32)), _p(out))
    return out


def dequant_value(codes, norm, Rm):
    out = np.empty(D, np.float64)
    lib().okqo_dequant_value(_p(_c(codes, np.uint8)), C.c_uint16(int(norm)), _p(_c(Rm, np.float32)), _p(out))
    return out


def unpack_codes(codes: np.ndarray) -> np.ndarray:
    """uint8 [..., 32] -> uint8 [..., 128] (pure bit plumbing, for the tests)."""
    codes = np.asarray(codes, np.uint8)
    sh = np.arange(4, dtype=np.uint8) * 2
    return ((codes[..., :, None] >> sh) & 3).reshape(*codes.shape[:-1], D)


def attention(path: int, q_bits, kq, vq, modality, k_tail, v_tail, signs, R, sm_scale=None,
              unit_seq=None, unit_rot=None):
    """Attention over U units.

    q_bits [U,G,128] u16; kq/vq dicts with arrays stacked over units ([U,np,32], [U,np], [U,np/32,128,2]);
    modality [S, >=n_total] u8; k_tail/v_tail [U,n_tail,128] u16 (n_tail <= 32).
    signs [nR,128], R [nR,3,128,128].  Returns (out float64 [U,G,128], threads used).
    """
    q_bits = _c(q_bits, np.uint16)
    U, G, _ = q_bits.shape
    kc = _c(kq["codes"], np.uint8); kn = _c(kq["norm"], np.uint16); km = _c(kq["meta"], np.uint16)
    vc = _c(vq["codes"], np.uint8); vn = _c(vq["norm"], np.uint16)
    npk = kc.shape[1]
    assert kc.shape == (U, npk, 32) and vc.shape == (U, npk, 32)
    modality = _c(modality, np.uint8)
    assert modality.max(initial=0) <= 2, "modality ids are 0 text, 1 audio, 2 video"
    if modality.ndim == 1:
        modality = modality[None]
    k_tail = _c(k_tail, np.uint16); v_tail = _c(v_tail, np.uint16)
    n_tail = k_tail.shape[1]
    assert n_tail <= W
    kt = np.zeros((U, W, D), np.uint16); vt = np.zeros((U, W, D), np.uint16)
    kt[:, :n_tail] = k_tail; vt[:, :n_tail] = v_tail
    signs = _c(signs, np.float32).reshape(-1, D)
    R = _c(R, np.float32).reshape(-1, 3, D, D)
    unit_seq = _c(np.zeros(U) if unit_seq is None else unit_seq, np.int32)
    unit_rot = _c(np.zeros(U) if unit_rot is None else unit_rot, np.int32)
    assert modality.shape[1] >= npk
    out = np.empty((U, G, D), np.float64)
    scale = 1.0 / np.sqrt(D) if sm_scale is None else sm_scale
    th = lib().okqo_attention_batch(C.c_int(path), C.c_int(U), _p(q_bits), C.c_int(G), C.c_int64(npk),
                                    _p(kc), _p(kn), _p(km), _p(vc), _p(vn), _p(modality),
                                    C.c_int64(modality.shape[1]), _p(unit_seq), _p(unit_rot), C.c_int(n_tail),
                                    _p(kt), _p(vt), _p(signs), _p(R), C.c_double(scale), _p(out))
    return out, th


def quantize_batch(k_bits, v_bits, modality, signs, R, unit_seq=None, unit_rot=None, meta_format=0):
    """k_bits, v_bits [U,n,128] u16 -> (kq, vq) stacked dicts, threads used.
    meta_format 1 = MXFP4 metadata: kq["meta"] holds the decoded (m', s') and kq["mx"] the stored bytes."""
    k_bits = _c(k_bits, np.uint16); v_bits = _c(v_bits, np.uint16)
    U, n, _ = k_bits.shape
    npk = (n // W) * W
    modality = _c(modality, np.uint8)
    assert modality.max(initial=0) <= 2, "modality ids are 0 text, 1 audio, 2 video"
    if modality.ndim == 1:
        modality = modality[None]
    signs = _c(signs, np.float32).reshape(-1, D)
    R = _c(R, np.float32).reshape(-1, 3, D, D)
    unit_seq = _c(np.zeros(U) if unit_seq is None else unit_seq, np.int32)
    unit_rot = _c(np.zeros(U) if unit_rot is None else unit_rot, np.int32)
    kq = {"codes": np.zeros((U, npk, 32), np.uint8), "norm": np.zeros((U, npk), np.uint16),
          "meta": np.zeros((U, npk // W, D, 2), np.uint16)}
    vq = {"codes": np.zeros((U, npk, 32), np.uint8), "norm": np.zeros((U, npk), np.uint16)}
    mx = np.zeros((U, npk // W, 136), np.uint8)
    th = lib().okqo_quantize_batch_fmt(C.c_int(U), _p(k_bits), _p(v_bits), C.c_int64(n), _p(modality),
                                       C.c_int64(modality.shape[1]), _p(unit_seq), _p(unit_rot), _p(signs), _p(R),
                                       _p(kq["codes"]), _p(kq["norm"]), _p(kq["meta"]), _p(vq["codes"]), _p(vq["norm"]),
                                       C.c_int(meta_format), _p(mx))
    if meta_format == 1:
        kq["mx"] = mx
    return kq, vq, th


# ---------------------------------------------------------------- streaming schedules

def packed_counts(n: int, schedule: int):
    """(packed keys, packed values) of a sequence of n tokens.

    schedule 0: both are packed as soon as a 32-token window is complete.
    schedule 1, the paper's captioning schedule (Implementation details): keys are quantised every 128 tokens,
    in groups of 32; values stay behind a 128-token sliding fp16 window before they are quantised (window by
    window, since a value record holds 32 tokens)."""
    if schedule == 0:
        return (n // W) * W, (n // W) * W
    return (n // 128) * 128, (((n - 128) // W) * W if n >= 128 else 0)


def attention_scheduled(q_bits, kq, vq, modality, k_bits, v_bits, signs, R, k_packed: int, v_packed: int,
                        sm_scale=None):
    """Attention of one (layer, sequence, KV head) by definition, in fp64, when the first `k_packed` keys and the
    first `v_packed` values are read from the packed cache and the rest are still raw fp16:
    out_h = softmax(q_h K_hat^T * scale) V_hat with K_hat / V_hat the dequantised (Eq. 2-4, Eq. 6) or raw rows.

    q_bits [G,128] u16; kq / vq: one unit's packed arrays (codes [np,32], norm [np], meta [np/32,128,2]);
    modality [n] u8; k_bits / v_bits [n,128] u16 raw tokens.  Returns fp64 [G,128]."""
    k = half_to_float(_c(k_bits, np.uint16)).astype(np.float64).reshape(-1, D)
    v = half_to_float(_c(v_bits, np.uint16)).astype(np.float64).reshape(-1, D)
    for t in range(k_packed):
        k[t] = dequant_key(kq["codes"][t], kq["norm"][t], kq["meta"][t // W], signs)
    for t in range(v_packed):
        v[t] = dequant_value(vq["codes"][t], vq["norm"][t], R[int(modality[t])])
    q = half_to_float(_c(q_bits, np.uint16)).astype(np.float64).reshape(-1, D)
    scale = D ** -0.5 if sm_scale is None else sm_scale
    s = (q @ k.T) * scale
    s -= s.max(axis=1, keepdims=True)
    p = np.exp(s)
    return (p / p.sum(axis=1, keepdims=True)) @ v
