"""CPU oracle of the offline calibration of the per-modality value rotations (test infrastructure only:
imported by the tests alone, never by the product package).

Plain numpy in fp64, following the paper's "Modality-aware value rotation" paragraph:

  * attention weights of the calibration tokens, alpha[i, j] = softmax_j(q_i . k_j * scale);
  * value weights  w_j = sum_i alpha[i, j]^2                                   (Eq. 5, left);
  * per-modality weighted second moment  C_m = sum_{j in m} w_j v_j^T v_j      (Eq. 5, right);
  * U_m = eigenvectors of C_m; the rotation that replaces z = H u is  R_m = H U_m^T.

Readings where the paper is silent (listed in the design notes as well):
  * alpha is the causal attention of a decoder (query i sees keys j <= i); `causal=False` gives the full
    softmax for the closed-form pins;
  * the sum over i runs over all query heads of the GQA group that share the KV head;
  * v_j is the raw value vector (not normalised);
  * eigenvectors are ordered by descending eigenvalue, each with its largest-magnitude component positive
    (any order / sign gives an equally valid orthogonal R_m);
  * H is the randomised Hadamard matrix of the key path, H = Had_128 diag(signs) / sqrt(128).

parity pins: closed forms (uniform and one-hot attention, an orthogonal value set, a diagonal moment
matrix), orthogonality of R_m, and the property the calibration exists for: on data with a
modality-specific low-rank structure the matched rotation gives the smallest 2-bit reconstruction error.
"""
from __future__ import annotations

import numpy as np

D = 128


def half_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def hadamard_matrix(signs: np.ndarray) -> np.ndarray:
    """H = Had_128 diag(signs) / sqrt(128) in fp64 (Sylvester order, the order the key path's transform uses)."""
    h = np.array([[1.0]])
    while h.shape[0] < D:
        h = np.block([[h, h], [h, -h]])
    return h * np.asarray(signs, dtype=np.float64)[None, :] / np.sqrt(float(D))


def attention_weights(q_bits: np.ndarray, k_bits: np.ndarray, sm_scale: float | None = None,
                      causal: bool = True) -> np.ndarray:
    """w_j = sum over heads g and queries i of alpha[g, i, j]^2.

    q_bits: uint16 [G, n, 128] (fp16 bit patterns), k_bits: uint16 [n, 128].  Returns fp64 [n]."""
    q = half_bits_to_f64(q_bits)
    k = half_bits_to_f64(k_bits)
    G, n, _ = q.shape
    scale = D ** -0.5 if sm_scale is None else sm_scale
    w = np.zeros(n, dtype=np.float64)
    for g in range(G):
        s = (q[g] @ k.T) * scale                       # [i, j]
        if causal:
            s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        alpha = p / p.sum(axis=1, keepdims=True)
        w += (alpha * alpha).sum(axis=0)
    return w


def weighted_moments(v_bits: np.ndarray, w: np.ndarray, modality: np.ndarray) -> np.ndarray:
    """C_m = sum_{j: modality_j = m} w_j v_j^T v_j for m = 0, 1, 2 (ids > 2 count as text, 0).  fp64 [3, 128, 128]."""
    v = half_bits_to_f64(v_bits)
    mod = np.asarray(modality).astype(np.int64)
    mod = np.where(mod > 2, 0, mod)
    C = np.zeros((3, D, D), dtype=np.float64)
    for m in range(3):
        sel = mod == m
        if sel.any():
            vm = v[sel]
            C[m] = (vm * np.asarray(w, dtype=np.float64)[sel, None]).T @ vm
    return C


def eigenbasis(Cm: np.ndarray):
    """Eigenvalues (descending) and eigenvectors (columns) of a symmetric matrix, each eigenvector with its
    largest-magnitude component positive."""
    lam, U = np.linalg.eigh(np.asarray(Cm, dtype=np.float64))
    order = np.argsort(-lam, kind="stable")
    lam, U = lam[order], U[:, order]
    piv = np.abs(U).argmax(axis=0)
    U = U * np.where(U[piv, np.arange(U.shape[1])] < 0, -1.0, 1.0)[None, :]
    return lam, U


def rotation_from_moment(Cm: np.ndarray, signs: np.ndarray):
    """R_m = H U_m^T (so that z = R_m u = H (U_m^T u)) and the eigenvalues.  fp64."""
    lam, U = eigenbasis(Cm)
    return hadamard_matrix(signs) @ U.T, lam


def calibrate(q_bits, k_bits, v_bits, modality, signs, sm_scale=None, causal=True):
    """The whole calibration of one (layer, KV head): returns (w, C [3,128,128], R [3,128,128], lam [3,128])."""
    w = attention_weights(q_bits, k_bits, sm_scale, causal)
    C = weighted_moments(v_bits, w, modality)
    R = np.zeros((3, D, D)); lam = np.zeros((3, D))
    for m in range(3):
        R[m], lam[m] = rotation_from_moment(C[m], signs)
    return w, C, R, lam
