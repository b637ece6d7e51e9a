"""Pins of the calibration oracle (Eq. 5 and R_m = H U_m^T) against closed forms, invariants and the
property the calibration exists for.  CPU only."""
import numpy as np
import pytest

from oracle import okq_calib_oracle as CO
from oracle import okq_oracle as O
from paper_2609_11582_b200 import workloads as WL

D = 128


def f16bits(x):
    return np.asarray(x, dtype=np.float16).view(np.uint16)


def test_hadamard_matrix_is_the_key_path_transform():
    rng = np.random.default_rng(1)
    signs = np.where(rng.random(D) < 0.5, -1.0, 1.0).astype(np.float32)
    H = CO.hadamard_matrix(signs)
    assert np.allclose(H @ H.T, np.eye(D), atol=1e-12)
    x = rng.standard_normal(D).astype(np.float32)
    # the C oracle's in-place butterflies (stages h = 1 .. 64) on diag(signs) x, scaled by 1/sqrt(128)
    ref = O.fwht128((signs * x).astype(np.float32)).astype(np.float64) / np.sqrt(128.0)
    assert np.allclose(H @ x.astype(np.float64), ref, rtol=0, atol=1e-5)


def test_uniform_attention_closed_forms():
    G, n = 3, 37
    q = np.zeros((G, n, D), np.float16).view(np.uint16)       # all scores equal
    k = f16bits(np.random.default_rng(2).standard_normal((n, D)))
    w = CO.attention_weights(q, k, causal=False)
    assert np.allclose(w, G / n, rtol=1e-12)                  # alpha = 1/n: sum_i (1/n)^2 = 1/n per head
    w = CO.attention_weights(q, k, causal=True)
    ref = np.array([sum(1.0 / (i + 1) ** 2 for i in range(j, n)) for j in range(n)]) * G
    assert np.allclose(w, ref, rtol=1e-12)                    # alpha[i, j] = 1/(i+1) for j <= i


def test_one_hot_attention_counts_queries():
    n = 16
    k = np.zeros((n, D), np.float16)
    k[np.arange(n), np.arange(n)] = 64.0                       # orthogonal keys, large: softmax is one-hot
    target = np.array([3, 3, 7, 0, 3, 15, 7, 7, 1, 0, 0, 3, 12, 12, 12, 3])
    q = np.zeros((1, n, D), np.float16)
    q[0, np.arange(n), target] = 64.0
    w = CO.attention_weights(q.view(np.uint16), k.view(np.uint16), sm_scale=1.0, causal=False)
    assert np.allclose(w, np.bincount(target, minlength=n), atol=1e-9)


def test_weighted_moments_closed_forms():
    rng = np.random.default_rng(3)
    n = 50
    v = rng.standard_normal((n, D)).astype(np.float16)
    w = rng.random(n)
    mod = rng.integers(0, 4, n)                                # id 3 counts as text
    C = CO.weighted_moments(v.view(np.uint16), w, mod)
    v64 = v.astype(np.float64)
    total = sum(w[j] * np.outer(v64[j], v64[j]) for j in range(n))
    assert np.allclose(C.sum(axis=0), total, rtol=1e-12, atol=1e-12)
    for m in range(3):
        sel = np.where(mod > 2, 0, mod) == m
        assert np.allclose(np.trace(C[m]), (w[sel] * (v64[sel] ** 2).sum(axis=1)).sum(), rtol=1e-12)
        assert np.allclose(C[m], C[m].T, atol=0)
    # scaled unit vectors: a diagonal moment matrix with the weights on the diagonal
    e = np.zeros((4, D), np.float16); idx = [5, 17, 17, 100]; e[np.arange(4), idx] = [1, 2, 1, 0.5]
    C = CO.weighted_moments(e.view(np.uint16), np.array([1.0, 0.25, 3.0, 8.0]), np.zeros(4, np.int64))
    d = np.zeros(D); d[5] = 1.0; d[17] = 0.25 * 4 + 3.0; d[100] = 8 * 0.25
    assert np.allclose(C[0], np.diag(d)) and not C[1].any() and not C[2].any()


def test_eigenbasis_and_rotation_invariants():
    rng = np.random.default_rng(4)
    lam_true = np.sort(rng.random(D) + 0.1)[::-1] * np.arange(D, 0, -1)
    Q, _ = np.linalg.qr(rng.standard_normal((D, D)))
    C = (Q * lam_true) @ Q.T
    lam, U = CO.eigenbasis(C)
    assert np.allclose(lam, lam_true, rtol=1e-10)
    assert np.allclose(U.T @ U, np.eye(D), atol=1e-12)
    assert np.allclose(C @ U, U * lam, atol=1e-9 * lam_true[0])
    assert (U[np.abs(U).argmax(axis=0), np.arange(D)] > 0).all()
    assert np.allclose(np.abs(U.T @ Q), np.eye(D), atol=1e-8)          # the planted eigenvectors, up to sign
    lam_d, U_d = CO.eigenbasis(np.diag(np.arange(1.0, D + 1)))          # diagonal: a permutation
    assert np.allclose(lam_d, np.arange(D, 0, -1)) and np.allclose(U_d, np.eye(D)[:, ::-1])
    signs = np.where(rng.random(D) < 0.5, -1.0, 1.0)
    R, lam_r = CO.rotation_from_moment(C, signs)
    H = CO.hadamard_matrix(signs)
    assert np.allclose(R @ R.T, np.eye(D), atol=1e-12)
    assert np.allclose(R @ C @ R.T, (H * lam_r) @ H.T, atol=1e-9 * lam_true[0])
    # in the rotated basis every coordinate carries the same share of the weighted energy
    assert np.allclose(np.diag(R @ C @ R.T), lam_true.sum() / D, rtol=1e-9)


def _recon_mse(v_bits, R32):
    """Relative reconstruction error of the 2-bit value quantiser (Eq. 6: x_hat = norm * R^T cb[code])."""
    mod = np.zeros(v_bits.shape[0], np.uint8)
    vq = O.quantize_values(v_bits, mod, np.stack([R32, R32, R32]))
    levels, _ = O.codebook()
    z_hat = np.asarray(levels, dtype=np.float64)[O.unpack_codes(vq["codes"])]          # [n, 128]
    rec = (z_hat @ R32.astype(np.float64)) * O.half_to_float(vq["norm"]).astype(np.float64)[:, None]
    v = v_bits.view(np.float16).astype(np.float64)[: rec.shape[0]]       # whole 32-token windows only
    return float(((rec - v) ** 2).sum() / (v ** 2).sum())


def test_matched_rotation_gives_the_lowest_error():
    """Values of each modality live near their own 16-dimensional subspace (the synthetic workload's recipe).
    Quantising them with the rotation calibrated on the same modality gives a smaller reconstruction error
    than with another modality's rotation, a rotation calibrated on the pooled data, or the plain Hadamard."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=1, n_tokens=4096)
    _, v = WL.gen_kv(w, 0, n_tokens=4096)
    mod = WL.modality_layout(w, 4096).numpy()
    vb = v[0, 0].numpy().view(np.uint16)                                 # one KV head: [n, 128]
    signs = WL.gen_signs(w, 0).numpy()
    ones = np.ones(vb.shape[0])
    C = CO.weighted_moments(vb, ones, mod)
    R = [CO.rotation_from_moment(C[m], signs)[0].astype(np.float32) for m in range(3)]
    R_pool = CO.rotation_from_moment(C.sum(axis=0), signs)[0].astype(np.float32)
    H = CO.hadamard_matrix(signs).astype(np.float32)
    for m in range(3):
        vm = np.ascontiguousarray(vb[mod == m])
        matched = _recon_mse(vm, R[m])
        others = {f"modality {o}": _recon_mse(vm, R[o]) for o in range(3) if o != m}
        others["pooled"] = _recon_mse(vm, R_pool)
        others["hadamard"] = _recon_mse(vm, H)
        print(f"modality {m}: matched {matched:.4f}", {k: round(x, 4) for k, x in others.items()})
        assert all(matched < x for x in others.values()), (m, matched, others)
