"""CPU oracle for the bit-width ladder (K2V2 / K3V3 / K4V4) and for the TurboQuant baseline codec.

TEST INFRASTRUCTURE ONLY: imported by tests/ (and by nothing in the product path).  Plain numpy, one
step per line, in the precision of the 2-bit oracle: rotated coordinates in fp32 (taken from the C
oracle's okqo_key_rotate / okqo_value_rotate, which are pinned on their own), code assignment in fp32,
reconstruction and error metrics in fp64.

What it computes
  * lloyd_max(bits): the 2^bits-level minimum-MSE quantiser of N(0, 1) (Eq. 3: "fixed codebook constructed
    from the Gaussian reference distribution"), by the fixed-point iteration level = mean of its cell,
    threshold = mid-point of neighbouring levels.  Pinned to Max's 1960 table for 4, 8 and 16 levels.
  * TurboQuant (Preliminaries, Eq. 2-3): norm, randomised Hadamard rotation, nearest level of the fixed
    codebook scaled to N(0, 1/128); the same for keys and values, no window statistics, no modality rotation.
  * OmniKVQuant at b bits: keys by Eq. 4 with 2^b uniform levels between the window's per-channel minimum and
    maximum (step = range / (2^b - 1), (m, s) stored as fp16, codes against the stored pair: the reading the
    2-bit oracle takes, with 3 replaced by 2^b - 1); values by Eq. 6 with the 2^b-level codebook.
  * storage rates in bits per element (the Bits/elem column of the error-comparison table).
At b = 2 the key and value codes equal the C oracle's bit for bit (pinned)."""
from __future__ import annotations

import numpy as np
from scipy.stats import norm as _gauss

from oracle import okq_oracle as O

D, W = 128, 32


# ---------------------------------------------------------------- codebooks (Eq. 3)
def lloyd_max(bits: int, iters: int = 2000):
    """(levels[2^bits], thresholds[2^bits - 1]) of the minimum-MSE quantiser of N(0, 1), fp64."""
    n = 1 << bits
    lv = np.linspace(-2.0, 2.0, n)
    for _ in range(iters):
        t = np.concatenate([[-np.inf], (lv[:-1] + lv[1:]) / 2, [np.inf]])
        new = (_gauss.pdf(t[:-1]) - _gauss.pdf(t[1:])) / (_gauss.cdf(t[1:]) - _gauss.cdf(t[:-1]))   # cell means
        if np.abs(new - lv).max() < 1e-15:
            lv = new
            break
        lv = new
    lv = (lv - lv[::-1]) / 2          # the quantiser of a symmetric density is symmetric: the middle threshold is exactly 0
    return lv, (lv[:-1] + lv[1:]) / 2


def lloyd_max_distortion(bits: int) -> float:
    """E (x - Q(x))^2 for x ~ N(0, 1): 1 - sum_cells P(cell) level^2 (levels are the cell means)."""
    lv, th = lloyd_max(bits)
    t = np.concatenate([[-np.inf], th, [np.inf]])
    return float(1.0 - ((_gauss.cdf(t[1:]) - _gauss.cdf(t[:-1])) * lv ** 2).sum())


def codebook32(bits: int):
    """The codebook of a unit vector's rotated coordinates, N(0, 1/128), as the fp32 constants a kernel holds."""
    lv, th = lloyd_max(bits)
    return (lv / np.sqrt(D)).astype(np.float32), (th / np.sqrt(D)).astype(np.float32)


def codebook_codes(z: np.ndarray, bits: int) -> np.ndarray:
    """Nearest level = number of thresholds below z (a value on a threshold takes the lower code); z fp32 [..]."""
    _, th = codebook32(bits)
    return (z[..., None] > th).sum(axis=-1).astype(np.uint8)


# ---------------------------------------------------------------- rotations (Eq. 2, Eq. 6): the 2-bit oracle's
def rotate_keys(k_bits: np.ndarray, signs: np.ndarray):
    """k_bits u16 [n,128] -> (norm bits u16 [n], z fp32 [n,128] = H k / fp16(||k||))."""
    out = [O.key_rotate(np.ascontiguousarray(row), signs) for row in k_bits]
    return np.array([o[0] for o in out], dtype=np.uint16), np.stack([o[1] for o in out]).astype(np.float32)


def rotate_values(v_bits: np.ndarray, modality: np.ndarray, R: np.ndarray):
    """v_bits u16 [n,128], modality u8 [n] (ids > 2 count as text), R fp32 [3,128,128] -> (norm bits, z = R_m v / norm)."""
    mod = np.where(modality > 2, 0, modality)
    out = [O.value_rotate(np.ascontiguousarray(row), R[int(m)]) for row, m in zip(v_bits, mod)]
    return np.array([o[0] for o in out], dtype=np.uint16), np.stack([o[1] for o in out]).astype(np.float32)


def hadamard_matrix(signs: np.ndarray) -> np.ndarray:
    """H = Had_128 diag(signs) / sqrt(128), Sylvester order, fp64 (H H^T = I)."""
    h = np.array([[1.0]])
    while h.shape[0] < D:
        h = np.block([[h, h], [h, -h]])
    return h * signs.astype(np.float64)[None, :] / np.sqrt(D)


# ---------------------------------------------------------------- TurboQuant (Preliminaries)
def turboquant_encode(x_bits: np.ndarray, signs: np.ndarray, bits: int):
    """x_bits u16 [n,128] -> (codes u8 [n,128], norm bits u16 [n]): Eq. 2 then Eq. 3."""
    norm, z = rotate_keys(x_bits, signs)
    return codebook_codes(z, bits), norm


def turboquant_decode(codes: np.ndarray, norm_bits: np.ndarray, signs: np.ndarray, bits: int) -> np.ndarray:
    """x_hat = ||x|| H^T cb[codes], fp64 [n,128]."""
    lv, _ = codebook32(bits)
    nrm = O.half_to_float(norm_bits).astype(np.float64)
    return (lv.astype(np.float64)[codes] @ hadamard_matrix(signs)) * nrm[:, None]


# ---------------------------------------------------------------- OmniKVQuant keys at b bits (Eq. 4)
def key_window_quantize(z: np.ndarray, bits: int):
    """z fp32 [32,128] -> (meta u16 [128,2] = fp16 (m, s), codes u8 [32,128]).  fp32, every operation rounded."""
    L = np.float32((1 << bits) - 1)
    z = z.astype(np.float32)
    mn, mx = z.min(axis=0), z.max(axis=0)
    m_h = O.float_to_half(mn)
    m_f = O.half_to_float(m_h).astype(np.float32)
    rng = np.maximum(mx - m_f, np.float32(0.0)).astype(np.float32)       # m rounded up past a (near-)constant channel
    s_h = O.float_to_half((rng / L).astype(np.float32))
    s_f = O.half_to_float(s_h).astype(np.float32)
    live = s_f > 0
    r = np.where(live, np.float32(1.0) / np.where(live, s_f, np.float32(1.0)), np.float32(0.0)).astype(np.float32)
    q = np.rint(((z - m_f[None, :]).astype(np.float32) * r[None, :]).astype(np.float32))   # round-half-even
    codes = np.where(live[None, :], np.clip(q, 0, float(L)), 0).astype(np.uint8)
    return np.stack([m_h, s_h], axis=1).astype(np.uint16), codes


def quantize_keys(k_bits: np.ndarray, signs: np.ndarray, bits: int):
    """k_bits u16 [n,128], n a multiple of 32 -> dict(codes u8 [n,128], norm u16 [n], meta u16 [n/32,128,2])."""
    norm, z = rotate_keys(k_bits, signs)
    metas, codes = [], []
    for g in range(z.shape[0] // W):
        m, c = key_window_quantize(z[g * W:(g + 1) * W], bits)
        metas.append(m); codes.append(c)
    return {"codes": np.concatenate(codes), "norm": norm, "meta": np.stack(metas)}


def dequant_keys(kq: dict, signs: np.ndarray) -> np.ndarray:
    """k_hat = ||k|| H^T (m + s code), fp64 [n,128]."""
    shape = kq["meta"].shape[:2]
    m = O.half_to_float(kq["meta"][..., 0]).astype(np.float64).reshape(shape)
    s = O.half_to_float(kq["meta"][..., 1]).astype(np.float64).reshape(shape)
    zh = np.repeat(m, W, axis=0) + np.repeat(s, W, axis=0) * kq["codes"].astype(np.float64)
    return (zh @ hadamard_matrix(signs)) * O.half_to_float(kq["norm"]).astype(np.float64)[:, None]


# ---------------------------------------------------------------- OmniKVQuant values at b bits (Eq. 6, Eq. 3)
def quantize_values(v_bits: np.ndarray, modality: np.ndarray, R: np.ndarray, bits: int):
    norm, z = rotate_values(v_bits, modality, R)
    return {"codes": codebook_codes(z, bits), "norm": norm}


def dequant_values(vq: dict, modality: np.ndarray, R: np.ndarray, bits: int) -> np.ndarray:
    """v_hat = ||v|| R_m^T cb[codes], fp64 [n,128]."""
    lv, _ = codebook32(bits)
    mod = np.where(modality > 2, 0, modality)
    zh = lv.astype(np.float64)[vq["codes"]]
    out = np.einsum("nc,ncd->nd", zh, R.astype(np.float64)[mod])
    return out * O.half_to_float(vq["norm"]).astype(np.float64)[:, None]


# ---------------------------------------------------------------- storage (Bits/elem column)
def bits_per_element(k_bits: int, v_bits: int, meta: str) -> float:
    """Average over K and V of: code bits + fp16 norm per 128-vector + key (m, s) metadata per 32-token window.
    meta: 'none' (TurboQuant), 'fp16', 'mxfp4' (4-bit elements + one 8-bit scale per 32)."""
    per_pair = {"none": 0.0, "fp16": 2 * 16.0, "mxfp4": 2 * (4.0 + 8.0 / 32)}[meta]
    return ((k_bits + 16.0 / D + per_pair / W) + (v_bits + 16.0 / D)) / 2
