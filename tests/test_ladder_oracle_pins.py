"""Pins of the bit-width-ladder oracle (oracle/okq_ladder_oracle.py: 3- and 4-bit codes, TurboQuant codec) against
what the paper and the mathematics fix: Max's 1960 table, the Lloyd-Max fixed-point equations by numerical
integration, brute-force nearest-level search, the 2-bit C oracle bit for bit at b = 2, exact-reconstruction and
error-bound cases of the window quantiser, textbook distortions on Gaussian vectors, the storage rates the paper's
error table prints, and the ordering of its bit-width ladder table (OmniKVQuant below TurboQuant at every width).  CPU only."""
import os

import numpy as np
import pytest
from scipy import integrate
from scipy.stats import norm as gauss

from oracle import okq_ladder_oracle as LO
from oracle import okq_oracle as O
from paper_2609_11582_b200 import workloads as WL

D, W = 128, 32
HERE = os.path.dirname(os.path.abspath(__file__))


def golden():
    out = {}
    for line in open(os.path.join(HERE, "golden", "lloyd_max_8_16level.txt")):
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            out[k] = np.array([float(x) for x in v])
    return out


def agrees(x, table):
    """Within one unit of the fourth significant digit, the precision the table prints (and was computed to in 1960)."""
    x, table = np.atleast_1d(x), np.atleast_1d(table)
    unit = 10.0 ** (np.floor(np.log10(np.abs(table))) - 3)
    return x.shape == table.shape and bool((np.abs(x - table) <= 1.001 * unit).all())


@pytest.mark.parametrize("bits,n", [(3, 8), (4, 16)])
def test_codebooks_are_max_1960_table(bits, n):
    g = golden()
    lv, th = LO.lloyd_max(bits)
    assert np.allclose(lv, -lv[::-1], atol=1e-12) and abs(th[n // 2 - 1]) < 1e-12          # symmetric, 0 a threshold
    assert agrees(lv[n // 2:], g[f"levels{n}"])
    assert agrees(th[n // 2:], g[f"thresholds{n}"])
    # the table's mean-squared errors come from a 1960 numerical integration: good to about three digits
    assert abs(LO.lloyd_max_distortion(bits) - g[f"distortion{n}"][0]) < 1e-3 * g[f"distortion{n}"][0]


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_codebooks_satisfy_the_fixed_point_equations(bits):
    """Each level is the conditional mean of N(0,1) on its cell (numerical integration), thresholds are mid-points,
    and the distortion equals the integral of (x - level)^2."""
    lv, th = LO.lloyd_max(bits)
    t = np.concatenate([[-12.0], th, [12.0]])
    dist = 0.0
    for i in range(len(lv)):
        mass = integrate.quad(gauss.pdf, t[i], t[i + 1])[0]
        mean = integrate.quad(lambda x: x * gauss.pdf(x), t[i], t[i + 1])[0] / mass
        assert abs(mean - lv[i]) < 1e-9
        dist += integrate.quad(lambda x: (x - lv[i]) ** 2 * gauss.pdf(x), t[i], t[i + 1])[0]
    assert np.allclose(th, (lv[:-1] + lv[1:]) / 2)
    assert abs(dist - LO.lloyd_max_distortion(bits)) < 1e-9


def test_two_bit_codebook_is_the_c_oracles():
    lv32, th32 = LO.codebook32(2)
    levels, thresh = O.codebook()
    assert np.array_equal(lv32, np.asarray(levels, np.float32)) and th32[2] == np.float32(thresh) and th32[1] == 0.0


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_threshold_counting_is_nearest_level(bits):
    rng = np.random.default_rng(bits)
    z = (rng.standard_normal(20000) / np.sqrt(D)).astype(np.float32)
    lv, th = LO.codebook32(bits)
    brute = np.abs(z[:, None].astype(np.float64) - lv.astype(np.float64)[None, :]).argmin(axis=1)
    keep = np.abs(z[:, None] - th[None, :]).min(axis=1) > 1e-7        # ties and near-ties aside
    assert np.array_equal(LO.codebook_codes(z, bits)[keep], brute[keep])
    assert LO.codebook_codes(th.copy(), bits).tolist() == list(range(len(th)))       # on a threshold: the lower code


@pytest.fixture(scope="module")
def data():
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=1, n_tokens=1024)
    k, v = WL.gen_kv(w, 0, n_tokens=1024)
    q = WL.gen_queries(w, 0)[0, : w.group].numpy().astype(np.float64)
    return (k[0, 0].numpy().view(np.uint16), v[0, 0].numpy().view(np.uint16), q, WL.gen_signs(w, 0).numpy(),
            WL.gen_rotations(w, 0).numpy(), WL.modality_layout(w, 1024).numpy())


def test_two_bits_equal_the_c_oracle_bit_for_bit(data):
    kb, vb, _, signs, R, mod = data
    kq, vq = LO.quantize_keys(kb, signs, 2), LO.quantize_values(vb, mod, R, 2)
    ck, cv = O.quantize_keys(kb, signs), O.quantize_values(vb, mod, R)
    assert np.array_equal(kq["norm"], ck["norm"]) and np.array_equal(kq["meta"], ck["meta"])
    assert np.array_equal(kq["codes"], O.unpack_codes(ck["codes"]))
    assert np.array_equal(vq["norm"], cv["norm"]) and np.array_equal(vq["codes"], O.unpack_codes(cv["codes"]))


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_window_quantiser_grid_is_reconstructed_exactly_and_error_is_bounded(bits):
    L = (1 << bits) - 1
    rng = np.random.default_rng(10 + bits)
    # channels on the grid m + s {0..L} with fp16-exact m, s whose products are fp32-exact: codes and values come back
    m = rng.integers(-64, 64, D).astype(np.float32) / 128.0
    s = rng.integers(1, 32, D).astype(np.float32) / 256.0
    codes = rng.integers(0, L + 1, (W, D))
    codes[0], codes[1] = 0, L                                   # every channel spans its full range
    z = (m[None, :] + s[None, :] * codes).astype(np.float32)
    meta, got = LO.key_window_quantize(z, bits)
    assert np.array_equal(got, codes)
    assert np.array_equal(O.half_to_float(meta[:, 0]), m) and np.array_equal(O.half_to_float(meta[:, 1]), s)
    # random data: |z_hat - z| <= s/2 + |m_h - min| + rounding of s (3 ulp of fp16), codes within range
    z = (rng.standard_normal((W, D)) * 0.09).astype(np.float32)
    meta, got = LO.key_window_quantize(z, bits)
    mf, sf = O.half_to_float(meta[:, 0]).astype(np.float64), O.half_to_float(meta[:, 1]).astype(np.float64)
    err = np.abs(mf[None, :] + sf[None, :] * got - z)
    bound = sf / 2 + np.abs(mf - z.min(axis=0)) + L * sf * 2.0 ** -10
    assert got.max() <= L and (err <= bound[None, :] + 1e-7).all()
    # a constant channel: s = 0, codes 0
    z[:, 5] = np.float32(0.25)
    meta, got = LO.key_window_quantize(z, bits)
    assert meta[5, 1] == 0 and (got[:, 5] == 0).all() and O.half_to_float(meta[5:6, 0])[0] == 0.25


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_gaussian_vectors_reach_the_textbook_distortion(bits):
    """Isotropic Gaussian vectors through a Haar rotation: relative reconstruction error -> the codebook's distortion
    (0.1175 / 0.03454 / 0.009497); and the TurboQuant codec, which is the same thing with the Hadamard rotation."""
    rng = np.random.default_rng(3)
    n = 512
    x = rng.standard_normal((n, D)).astype(np.float16)
    R = np.broadcast_to(WL.gen_rotations(WL.WORKLOADS["tiny"], 0).numpy()[0], (3, D, D)).copy()
    mod = np.zeros(n, np.uint8)
    xb = x.view(np.uint16)
    x64 = x.astype(np.float64)
    want = LO.lloyd_max_distortion(bits)
    vq = LO.quantize_values(xb, mod, R, bits)
    rel = ((LO.dequant_values(vq, mod, R, bits) - x64) ** 2).sum() / (x64 ** 2).sum()
    assert abs(rel - want) < 0.06 * want + 2e-4, (rel, want)
    signs = WL.gen_signs(WL.WORKLOADS["tiny"], 0).numpy()
    codes, norm = LO.turboquant_encode(xb, signs, bits)
    rel = ((LO.turboquant_decode(codes, norm, signs, bits) - x64) ** 2).sum() / (x64 ** 2).sum()
    assert abs(rel - want) < 0.06 * want + 2e-4, (rel, want)


def test_storage_rates():
    # the four values the error-comparison table prints
    assert LO.bits_per_element(2, 2, "none") == 2.125 and LO.bits_per_element(3, 2, "none") == 2.625
    assert LO.bits_per_element(2, 2, "fp16") == 2.625 and LO.bits_per_element(2, 2, "mxfp4") == 2.2578125
    # the ladder: one more bit per element on K and V each
    assert LO.bits_per_element(3, 3, "fp16") == 3.625 and LO.bits_per_element(4, 4, "mxfp4") == 4.2578125
    assert LO.bits_per_element(2, 2, "fp16") == O.bytes_per_token_head() * 8 / (2 * D)


def _softmax(s):
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    return p / p.sum(axis=-1, keepdims=True)


def test_ladder_ordering_on_the_synthetic_workload(data):
    """Bit-width ladder table: OmniKVQuant ahead of TurboQuant at K2V2, K3V3 and K4V4, both improving with the width.
    Re-run with key reconstruction error, attention KL and attention-output error on the synthetic cache."""
    kb, vb, q, signs, R, mod = data
    k = kb.view(np.float16).astype(np.float64)
    v = vb.view(np.float16).astype(np.float64)
    p = _softmax(q @ k.T / np.sqrt(D))

    def metrics(kh, vh):
        ph = _softmax(q @ kh.T / np.sqrt(D))
        return (((k - kh) ** 2).sum(axis=1).mean(), (p * (np.log(p + 1e-300) - np.log(ph + 1e-300))).sum(axis=1).mean(),
                (((p @ v) - (ph @ vh)) ** 2).sum(axis=1).mean())

    prev_o = prev_t = None
    for bits in (2, 3, 4):
        ours = metrics(LO.dequant_keys(LO.quantize_keys(kb, signs, bits), signs),
                       LO.dequant_values(LO.quantize_values(vb, mod, R, bits), mod, R, bits))
        tq = metrics(LO.turboquant_decode(*LO.turboquant_encode(kb, signs, bits), signs, bits),
                     LO.turboquant_decode(*LO.turboquant_encode(vb, signs, bits), signs, bits))
        print(f"K{bits}V{bits}: ours recon {ours[0]:.4f} KL {ours[1]:.5f} out {ours[2]:.6f} | TurboQuant {tq[0]:.4f} {tq[1]:.5f} {tq[2]:.6f}")
        assert ours[0] < tq[0] and ours[1] < tq[1]
        if prev_o is not None:
            assert ours[0] < prev_o[0] / 2.5 and tq[0] < prev_t[0] / 2.5        # about 4x per extra bit
            assert ours[1] < prev_o[1] and tq[1] < prev_t[1] and ours[2] < prev_o[2]
        prev_o, prev_t = ours, tq
