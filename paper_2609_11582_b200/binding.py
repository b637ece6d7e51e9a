"""Thin ctypes binding of the okq C ABI (argument marshalling only).

PyTorch is used for device memory and streams; every step of the path runs in the CUDA
library.  If the library is missing this module raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libokq.so")

HEAD_DIM, WINDOW, RECORD_BYTES, MAX_GROUP = 128, 32, 2688, 8
RECORD_BYTES_MX, MX_META_BYTES = 2312, 136
META_FP16, META_MXFP4 = 0, 1
SCHEDULE_WINDOW, SCHEDULE_CAPTION = 0, 1

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_CAPACITY, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(8)


class okq_cache(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("batch", C.c_int32), ("n_kv_heads", C.c_int32), ("n_q_heads", C.c_int32),
                ("head_dim", C.c_int32), ("window", C.c_int32), ("capacity", C.c_int32), ("meta_format", C.c_int32),
                ("schedule", C.c_int32), ("reserved", C.c_int32),
                ("records", C.c_void_p), ("modality", C.c_void_p), ("k_tail", C.c_void_p), ("v_tail", C.c_void_p),
                ("seq_len", C.c_void_p), ("status", C.c_void_p)]


class okq_ladder_cache(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_kv_heads", C.c_int32), ("n_q_heads", C.c_int32), ("capacity", C.c_int32),
                ("bits", C.c_int32), ("reserved", C.c_int32),
                ("k_codes", C.c_void_p), ("k_norm", C.c_void_p), ("k_meta", C.c_void_p), ("v_codes", C.c_void_p),
                ("v_norm", C.c_void_p), ("modality", C.c_void_p)]


class OkqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().okq_status_string(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError {lib().okq_last_cuda_error()})"
        super().__init__(f"{where}: {msg}")


_lib = None


def lib():
    """Load libokq.so (built in-tree by `python -m paper_2609_11582_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_11582_b200.build` "
                               "(the okq path has no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.okq_status_string.restype = C.c_char_p
        L.okq_status_string.argtypes = [C.c_int]
        L.okq_last_cuda_error.restype = C.c_int
        L.okq_cache_sizes.restype = C.c_int
        L.okq_cache_sizes.argtypes = [C.POINTER(okq_cache), C.POINTER(C.c_size_t)]
        L.okq_decode_workspace_bytes.restype = C.c_size_t
        L.okq_decode_workspace_bytes.argtypes = [C.POINTER(okq_cache), C.c_int32, C.c_int32]
        L.okq_quantize_keys.restype = C.c_int
        L.okq_quantize_keys.argtypes = [C.POINTER(okq_cache), C.c_int32, C.c_void_p, C.POINTER(C.c_int64), C.c_int32,
                                        C.c_void_p, C.c_void_p]
        L.okq_quantize_values.restype = C.c_int
        L.okq_quantize_values.argtypes = [C.POINTER(okq_cache), C.c_int32, C.c_void_p, C.POINTER(C.c_int64), C.c_int32,
                                          C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.okq_quantize_values_bulk.restype = C.c_int
        L.okq_quantize_values_bulk.argtypes = L.okq_quantize_values.argtypes
        L.okq_debug_bulk_timeout.restype = C.c_int
        L.okq_debug_bulk_timeout.argtypes = list(L.okq_quantize_values.argtypes[:-1]) + [C.c_int64, C.c_void_p]
        L.okq_append.restype = C.c_int
        L.okq_append.argtypes = [C.POINTER(okq_cache), C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                 C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.okq_decode_attention.restype = C.c_int
        L.okq_decode_attention.argtypes = [C.POINTER(okq_cache), C.c_int32, C.c_int32, C.c_void_p, C.c_float,
                                           C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t, C.c_int32,
                                           C.c_void_p, C.c_void_p]
        L.okq_decode_attention_simt.restype = C.c_int
        L.okq_decode_attention_simt.argtypes = L.okq_decode_attention.argtypes
        L.okq_decode_attention_noalloc.restype = C.c_int
        L.okq_decode_attention_noalloc.argtypes = [C.POINTER(okq_cache), C.c_int32, C.c_int32, C.c_void_p, C.c_float,
                                                   C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.okq_decode_select.restype = C.c_int32
        L.okq_decode_select.argtypes = [C.c_int32]
        L.okq_profile_events.restype = None
        L.okq_profile_events.argtypes = [C.c_void_p, C.c_void_p]
        L.okq_cache_export.restype = C.c_int
        L.okq_cache_export.argtypes = [C.POINTER(okq_cache), C.c_int32] + [C.c_void_p] * 6
        L.okq_cache_export_mx.restype = C.c_int
        L.okq_cache_export_mx.argtypes = [C.POINTER(okq_cache), C.c_int32] + [C.c_void_p] * 7
        L.okq_calib_workspace_bytes.restype = C.c_size_t
        L.okq_calib_workspace_bytes.argtypes = [C.c_int32, C.c_int32]
        L.okq_calib_attention_weights.restype = C.c_int
        L.okq_calib_attention_weights.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_int32,
                                                  C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.okq_calib_moments.restype = C.c_int
        L.okq_calib_moments.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t,
                                        C.c_void_p, C.c_void_p]
        L.okq_calib_rotation.restype = C.c_int
        L.okq_calib_rotation.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p]
        L.okq_cache_import.restype = C.c_int
        L.okq_cache_import.argtypes = [C.POINTER(okq_cache), C.c_int32] + [C.c_void_p] * 6
        L.okq_ladder_codebook.restype = C.c_int32
        L.okq_ladder_codebook.argtypes = [C.c_int32, C.POINTER(C.c_float), C.POINTER(C.c_float)]
        L.okq_ladder_quantize_keys.restype = C.c_int
        L.okq_ladder_quantize_keys.argtypes = [C.POINTER(okq_ladder_cache), C.c_void_p, C.POINTER(C.c_int64), C.c_int32,
                                               C.c_void_p, C.c_void_p]
        L.okq_ladder_quantize_values.restype = C.c_int
        L.okq_ladder_quantize_values.argtypes = [C.POINTER(okq_ladder_cache), C.c_void_p, C.POINTER(C.c_int64), C.c_int32,
                                                 C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.okq_ladder_decode_attention.restype = C.c_int
        L.okq_ladder_decode_attention.argtypes = [C.POINTER(okq_ladder_cache), C.c_int32, C.c_void_p, C.c_float, C.c_void_p,
                                                  C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.okq_turboquant_encode.restype = C.c_int
        L.okq_turboquant_encode.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.okq_turboquant_decode.restype = C.c_int
        L.okq_turboquant_decode.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def exported_symbols():
    return ["okq_status_string", "okq_last_cuda_error", "okq_cache_sizes", "okq_decode_workspace_bytes",
            "okq_quantize_keys", "okq_quantize_values", "okq_append", "okq_decode_attention", "okq_cache_export",
            "okq_cache_import", "okq_profile_events", "okq_decode_select", "okq_decode_attention_simt",
            "okq_decode_attention_noalloc", "okq_quantize_values_bulk", "okq_debug_bulk_timeout", "okq_cache_export_mx",
            "okq_calib_workspace_bytes", "okq_calib_attention_weights", "okq_calib_moments", "okq_calib_rotation",
            "okq_ladder_codebook", "okq_ladder_quantize_keys", "okq_ladder_quantize_values",
            "okq_ladder_decode_attention", "okq_turboquant_encode", "okq_turboquant_decode"]


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _check(st: int, where: str):
    if st != OK:
        raise OkqError(st, where)


def cache_sizes(n_layers, batch, n_kv_heads, n_q_heads, capacity, head_dim=HEAD_DIM, window=WINDOW,
                meta_format=META_FP16, schedule=SCHEDULE_WINDOW):
    shape = okq_cache(n_layers, batch, n_kv_heads, n_q_heads, head_dim, window, capacity, meta_format, schedule, 0)
    out = (C.c_size_t * 6)()
    _check(lib().okq_cache_sizes(C.byref(shape), out), "okq_cache_sizes")
    return list(out)


class Cache:
    """Device buffers of a 2-bit KV cache plus the C struct that describes them."""

    def __init__(self, n_layers, batch, n_kv_heads, n_q_heads, capacity, device="cuda", meta_format=META_FP16,
                 schedule=SCHEDULE_WINDOW):
        sizes = cache_sizes(n_layers, batch, n_kv_heads, n_q_heads, capacity, meta_format=meta_format, schedule=schedule)
        self.meta_format, self.schedule = meta_format, schedule
        self.n_layers, self.batch, self.n_kv_heads, self.n_q_heads, self.capacity = (
            n_layers, batch, n_kv_heads, n_q_heads, capacity)
        self.device = torch.device(device)
        self.records = torch.zeros(sizes[0], dtype=torch.uint8, device=device)
        self.modality = torch.zeros(sizes[1], dtype=torch.uint8, device=device)
        self.k_tail = torch.zeros(sizes[2] // 2, dtype=torch.float16, device=device)
        self.v_tail = torch.zeros(sizes[3] // 2, dtype=torch.float16, device=device)
        self.seq_len = torch.zeros(n_layers * batch, dtype=torch.int32, device=device)
        self.status = torch.zeros(4, dtype=torch.int32, device=device)
        self.c = okq_cache(n_layers, batch, n_kv_heads, n_q_heads, HEAD_DIM, WINDOW, capacity, meta_format, schedule, 0,
                           self.records.data_ptr(), self.modality.data_ptr(), self.k_tail.data_ptr(),
                           self.v_tail.data_ptr(), self.seq_len.data_ptr(), self.status.data_ptr())

    @property
    def group(self):
        return self.n_q_heads // self.n_kv_heads

    def packed_bytes(self, n_tokens):
        """Bytes of packed records a decode step over n_tokens per sequence must read."""
        return self.n_layers * self.batch * self.n_kv_heads * (n_tokens // WINDOW) * (
            RECORD_BYTES_MX if self.meta_format == META_MXFP4 else RECORD_BYTES)

    def device_status(self) -> int:
        return int(self.status[0].item())


def quantize_keys(cache: Cache, layer: int, k: torch.Tensor, signs: torch.Tensor, n_tokens=None, stream=None):
    """k: fp16 [batch, n_kv_heads, n, 128] (last dim contiguous); signs: float32 [128]."""
    assert k.dtype == torch.float16 and k.stride(3) == 1
    n = k.shape[2] if n_tokens is None else n_tokens
    strides = (C.c_int64 * 3)(k.stride(0), k.stride(1), k.stride(2))
    _check(lib().okq_quantize_keys(C.byref(cache.c), layer, _ptr(k), strides, n, _ptr(signs), _stream(stream)),
           "okq_quantize_keys")


def quantize_values(cache: Cache, layer: int, v: torch.Tensor, modality: torch.Tensor, R: torch.Tensor,
                    n_tokens=None, stream=None, bulk=False):
    """v: fp16 [batch, n_kv_heads, n, 128]; modality: uint8 [batch, n]; R: float32 [n_R, 3, 128, 128].
    bulk=True calls okq_quantize_values_bulk (tensor-core rotation)."""
    assert v.dtype == torch.float16 and v.stride(3) == 1 and modality.dtype == torch.uint8 and modality.is_contiguous()
    n = v.shape[2] if n_tokens is None else n_tokens
    assert modality.shape[-1] == n
    strides = (C.c_int64 * 3)(v.stride(0), v.stride(1), v.stride(2))
    n_R = R.shape[0] if R.dim() == 4 else 1
    fn = lib().okq_quantize_values_bulk if bulk else lib().okq_quantize_values
    _check(fn(C.byref(cache.c), layer, _ptr(v), strides, n, _ptr(modality), _ptr(R), n_R, _stream(stream)),
           "okq_quantize_values_bulk" if bulk else "okq_quantize_values")


def debug_bulk_timeout(cache: Cache, layer: int, v: torch.Tensor, modality: torch.Tensor, R: torch.Tensor,
                       limit_clocks: int = 20_000_000, stream=None):
    """okq_debug_bulk_timeout: the bulk value quantiser with its first tile withheld and every wait limited to
    `limit_clocks` SM clocks; the device status word becomes ERR_TIMEOUT (testing aid)."""
    strides = (C.c_int64 * 3)(v.stride(0), v.stride(1), v.stride(2))
    n_R = R.shape[0] if R.dim() == 4 else 1
    _check(lib().okq_debug_bulk_timeout(C.byref(cache.c), layer, _ptr(v), strides, v.shape[2], _ptr(modality), _ptr(R), n_R,
                                        limit_clocks, _stream(stream)), "okq_debug_bulk_timeout")


def append(cache: Cache, layer: int, layer_count: int, k_new, v_new, modality_new, signs, R, n_R=1, stream=None):
    _check(lib().okq_append(C.byref(cache.c), layer, layer_count, _ptr(k_new), _ptr(v_new), _ptr(modality_new),
                            _ptr(signs), _ptr(R), n_R, _stream(stream)), "okq_append")


def decode_workspace_bytes(cache: Cache, layer_count: int, num_splits: int = 0) -> int:
    return lib().okq_decode_workspace_bytes(C.byref(cache.c), layer_count, num_splits)


def decode_attention(cache: Cache, layer: int, layer_count: int, q, signs, R, workspace, out, n_R=1,
                     sm_scale=None, num_splits=0, stream=None, simt=False):
    """q: fp16 [layer_count, batch, n_q_heads, 128]; out: float32 same shape; workspace: uint8 device tensor.
    simt=True calls okq_decode_attention_simt (CUDA-core cross-check) instead."""
    scale = HEAD_DIM ** -0.5 if sm_scale is None else sm_scale
    fn = lib().okq_decode_attention_simt if simt else lib().okq_decode_attention
    _check(fn(C.byref(cache.c), layer, layer_count, _ptr(q), scale, _ptr(signs), _ptr(R), n_R,
                                      _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
                                      num_splits, _ptr(out), _stream(stream)), "okq_decode_attention")


def decode_attention_noalloc(cache: Cache, layer: int, layer_count: int, q, signs, R, out, n_R=1, sm_scale=None,
                             num_splits=0, stream=None):
    """okq_decode_attention_noalloc: same result as decode_attention, scratch held inside the library
    (64 MiB per GPU, shared by all calls on that GPU; overlapping calls race).  Allocates nothing."""
    scale = HEAD_DIM ** -0.5 if sm_scale is None else sm_scale
    _check(lib().okq_decode_attention_noalloc(C.byref(cache.c), layer, layer_count, _ptr(q), scale, _ptr(signs),
                                              _ptr(R), n_R, num_splits, _ptr(out), _stream(stream)),
           "okq_decode_attention_noalloc")


def decode_select(impl: int) -> int:
    """Choose the split-K kernel of later decode calls (0: tcgen05, 1: mma.sync warp pairs, the default); returns the previous choice."""
    return lib().okq_decode_select(impl)


def profile_events(before=None, after=None):
    """Record two torch.cuda.Event objects around the split-K kernel of later decode calls (None clears)."""
    lib().okq_profile_events(None if before is None else before.cuda_event, None if after is None else after.cuda_event)


def cache_export(cache: Cache, layer: int, stream=None):
    """Canonical arrays of one layer as a dict of device tensors."""
    B, H, cap, dev = cache.batch, cache.n_kv_heads, cache.capacity, cache.device
    out = {"k_codes": torch.empty(B, H, cap, 32, dtype=torch.uint8, device=dev),
           "k_norm": torch.empty(B, H, cap, dtype=torch.float16, device=dev),
           "k_meta": torch.empty(B, H, cap // WINDOW, HEAD_DIM, 2, dtype=torch.float16, device=dev),
           "v_codes": torch.empty(B, H, cap, 32, dtype=torch.uint8, device=dev),
           "v_norm": torch.empty(B, H, cap, dtype=torch.float16, device=dev)}
    if cache.meta_format == META_MXFP4:   # k_meta = decoded pairs, k_mx = the stored bytes
        out["k_mx"] = torch.empty(B, H, cap // WINDOW, MX_META_BYTES, dtype=torch.uint8, device=dev)
        _check(lib().okq_cache_export_mx(C.byref(cache.c), layer, _ptr(out["k_codes"]), _ptr(out["k_norm"]),
                                         _ptr(out["k_meta"]), _ptr(out["k_mx"]), _ptr(out["v_codes"]),
                                         _ptr(out["v_norm"]), _stream(stream)), "okq_cache_export_mx")
        return out
    _check(lib().okq_cache_export(C.byref(cache.c), layer, _ptr(out["k_codes"]), _ptr(out["k_norm"]),
                                  _ptr(out["k_meta"]), _ptr(out["v_codes"]), _ptr(out["v_norm"]), _stream(stream)),
           "okq_cache_export")
    return out


def cache_import(cache: Cache, layer: int, arrays: dict, stream=None):
    a = {k: v.contiguous() for k, v in arrays.items()}
    _check(lib().okq_cache_import(C.byref(cache.c), layer, _ptr(a["k_codes"]), _ptr(a["k_norm"]), _ptr(a["k_meta"]),
                                  _ptr(a["v_codes"]), _ptr(a["v_norm"]), _stream(stream)), "okq_cache_import")


# ---- offline calibration of the value rotations (okq_calib.h)

def calib_workspace(group: int, n: int, device="cuda") -> torch.Tensor:
    return torch.empty(lib().okq_calib_workspace_bytes(group, n), dtype=torch.uint8, device=device)


def calib_attention_weights(q, k, workspace, sm_scale=None, causal=True, stream=None):
    """q: fp16 [group, n, 128], k: fp16 [n, 128] (contiguous) -> w float32 [n]."""
    assert q.dtype == torch.float16 and k.dtype == torch.float16 and q.is_contiguous() and k.is_contiguous()
    group, n = q.shape[0], q.shape[1]
    w = torch.empty(n, dtype=torch.float32, device=q.device)
    scale = HEAD_DIM ** -0.5 if sm_scale is None else sm_scale
    _check(lib().okq_calib_attention_weights(_ptr(q), _ptr(k), group, n, scale, 1 if causal else 0, _ptr(workspace),
                                             workspace.numel(), _ptr(w), _stream(stream)), "okq_calib_attention_weights")
    return w


def calib_moments(v, w, modality, workspace, stream=None):
    """v: fp16 [n, 128], w: float32 [n], modality: uint8 [n] -> C float32 [3, 128, 128]."""
    assert v.dtype == torch.float16 and v.is_contiguous() and w.dtype == torch.float32 and modality.dtype == torch.uint8
    Cm = torch.empty(3, HEAD_DIM, HEAD_DIM, dtype=torch.float32, device=v.device)
    _check(lib().okq_calib_moments(_ptr(v), _ptr(w), _ptr(modality), v.shape[0], _ptr(workspace), workspace.numel(),
                                   _ptr(Cm), _stream(stream)), "okq_calib_moments")
    return Cm


def calib_rotation(Cm, signs, workspace, stream=None):
    """Cm: float32 [128, 128] symmetric, signs: float32 [128] -> (R float32 [128, 128], eigenvalues [128], sweeps)."""
    assert Cm.dtype == torch.float32 and Cm.is_contiguous() and signs.dtype == torch.float32
    R = torch.empty(HEAD_DIM, HEAD_DIM, dtype=torch.float32, device=Cm.device)
    lam = torch.empty(HEAD_DIM, dtype=torch.float32, device=Cm.device)
    sweeps = torch.zeros(1, dtype=torch.int32, device=Cm.device)
    _check(lib().okq_calib_rotation(_ptr(Cm), _ptr(signs), _ptr(workspace), workspace.numel(), _ptr(R), _ptr(lam),
                                    _ptr(sweeps), _stream(stream)), "okq_calib_rotation")
    return R, lam, sweeps


# ---------------------------------------------------------------- bit-width ladder (okq_ladder.h)
class LadderCache:
    """Device buffers of an okq_ladder_cache at `bits` bits per code (canonical layout, one layer)."""

    def __init__(self, batch, n_kv_heads, n_q_heads, capacity, bits, device="cuda"):
        self.bits, self.capacity = bits, capacity
        dev = torch.device(device)
        rows = (batch, n_kv_heads, capacity)
        self.k_codes = torch.zeros(rows + (16 * bits,), dtype=torch.uint8, device=dev)
        self.v_codes = torch.zeros(rows + (16 * bits,), dtype=torch.uint8, device=dev)
        self.k_norm = torch.zeros(rows, dtype=torch.float16, device=dev)
        self.v_norm = torch.zeros(rows, dtype=torch.float16, device=dev)
        self.k_meta = torch.zeros((batch, n_kv_heads, capacity // WINDOW, HEAD_DIM, 2), dtype=torch.float16, device=dev)
        self.modality = torch.zeros((batch, capacity), dtype=torch.uint8, device=dev)
        self.c = okq_ladder_cache(batch, n_kv_heads, n_q_heads, capacity, bits, 0, _ptr(self.k_codes), _ptr(self.k_norm),
                                  _ptr(self.k_meta), _ptr(self.v_codes), _ptr(self.v_norm), _ptr(self.modality))


def ladder_codebook(bits: int):
    """(levels, thresholds) the kernels hold for `bits`, as Python lists of floats."""
    lv, th = (C.c_float * 16)(), (C.c_float * 15)()
    n = lib().okq_ladder_codebook(bits, lv, th)
    if n == 0:
        raise OkqError(ERR_UNSUPPORTED, "okq_ladder_codebook")
    return list(lv)[:n], list(th)[:n - 1]


def ladder_quantize_keys(cache: LadderCache, k: torch.Tensor, signs: torch.Tensor, stream=None):
    assert k.dtype == torch.float16 and k.stride(3) == 1
    strides = (C.c_int64 * 3)(k.stride(0), k.stride(1), k.stride(2))
    _check(lib().okq_ladder_quantize_keys(C.byref(cache.c), _ptr(k), strides, k.shape[2], _ptr(signs), _stream(stream)),
           "okq_ladder_quantize_keys")


def ladder_quantize_values(cache: LadderCache, v: torch.Tensor, modality: torch.Tensor, R: torch.Tensor, stream=None):
    assert v.dtype == torch.float16 and v.stride(3) == 1 and modality.dtype == torch.uint8 and modality.is_contiguous()
    strides = (C.c_int64 * 3)(v.stride(0), v.stride(1), v.stride(2))
    n_R = R.shape[0] if R.dim() == 4 else 1
    _check(lib().okq_ladder_quantize_values(C.byref(cache.c), _ptr(v), strides, v.shape[2], _ptr(modality), _ptr(R), n_R,
                                            _stream(stream)), "okq_ladder_quantize_values")


def ladder_decode_attention(cache: LadderCache, n_tokens: int, q, signs, R, out, sm_scale=None, stream=None):
    """q: fp16 [batch, n_q_heads, 128]; out: float32 [batch, n_q_heads, 128]."""
    n_R = R.shape[0] if R.dim() == 4 else 1
    scale = HEAD_DIM ** -0.5 if sm_scale is None else sm_scale
    _check(lib().okq_ladder_decode_attention(C.byref(cache.c), n_tokens, _ptr(q), scale, _ptr(signs), _ptr(R), n_R,
                                             _ptr(out), _stream(stream)), "okq_ladder_decode_attention")


def turboquant_encode(x: torch.Tensor, signs: torch.Tensor, bits: int, stream=None):
    """x: fp16 [n, 128] contiguous -> (codes uint8 [n, 16 * bits], norms fp16 [n])."""
    assert x.dtype == torch.float16 and x.is_contiguous() and x.shape[-1] == HEAD_DIM
    n = x.numel() // HEAD_DIM
    codes = torch.empty((n, 16 * bits), dtype=torch.uint8, device=x.device)
    norms = torch.empty((n,), dtype=torch.float16, device=x.device)
    _check(lib().okq_turboquant_encode(_ptr(x), n, bits, _ptr(signs), _ptr(codes), _ptr(norms), _stream(stream)),
           "okq_turboquant_encode")
    return codes, norms


def turboquant_decode(codes: torch.Tensor, norms: torch.Tensor, signs: torch.Tensor, bits: int, stream=None):
    n = norms.numel()
    x_hat = torch.empty((n, HEAD_DIM), dtype=torch.float32, device=codes.device)
    _check(lib().okq_turboquant_decode(_ptr(codes), _ptr(norms), n, bits, _ptr(signs), _ptr(x_hat), _stream(stream)),
           "okq_turboquant_decode")
    return x_hat
