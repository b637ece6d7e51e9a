"""GPU parity tests: the CUDA library, called through its C ABI, against the CPU oracle on
the same seeded inputs.  Packed output is compared bit for bit; attention within 1e-3
relative L2 (whole tensor and worst single head vector) and 5e-3 max-abs."""
import numpy as np
import pytest
import torch

from oracle import okq_oracle as O
from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL
from tests import harness as Hn

pytestmark = pytest.mark.gpu
D, W = 128, 32


@pytest.fixture(scope="module")
def tiny():
    return Hn.Case(WL.WORKLOADS["tiny"])


@pytest.fixture(scope="module")
def layer7b_small():
    # 7B single-layer shape at 2048+19 tokens: several windows, mixed-modality windows, ragged tail
    return Hn.Case(WL.scaled(WL.WORKLOADS["layer7b"], batch=2), n_tokens=2048 + 19)


def test_library_loaded_and_symbols():
    L = B.lib()
    for s in B.exported_symbols():
        assert hasattr(L, s)


def test_quantize_tiny_bit_exact(tiny):
    kq, vq, _, _ = tiny.oracle_quantize(0)
    Hn.compare_cache(tiny, 0, tiny.gpu_export(0), kq, vq)
    assert tiny.cache.seq_len.cpu().tolist() == [2048]
    assert tiny.cache.device_status() == 0
    assert (tiny.cache.modality[:2048].cpu() == tiny.mod).all()


def test_quantize_ragged_bit_exact_and_tail(layer7b_small):
    c = layer7b_small
    kq, vq, kb, vb = c.oracle_quantize(0)
    Hn.compare_cache(c, 0, c.gpu_export(0), kq, vq)
    U = c.w.batch * c.w.n_kv_heads
    kt = Hn.u16(c.cache.k_tail).reshape(U, W, D)[:, :19]
    vt = Hn.u16(c.cache.v_tail).reshape(U, W, D)[:, :19]
    assert (kt == kb[:, 2048:]).all() and (vt == vb[:, 2048:]).all()
    assert c.cache.seq_len.cpu().tolist() == [2048 + 19] * c.w.batch


@pytest.mark.parametrize("simt", [False, True])
def test_decode_tiny_matches_oracle(tiny, simt):
    ref, _ = tiny.oracle_attention(0)
    got = tiny.gpu_decode(0, simt=simt)[0]
    print("errors (rel-L2, worst head, max-abs):", Hn.assert_attention_close(got, ref))


def test_decode_ragged_matches_oracle_and_definition(layer7b_small):
    c = layer7b_small
    ref, _ = c.oracle_attention(0, path=1)
    ref_def, _ = c.oracle_attention(0, path=0)
    assert np.abs(ref - ref_def).max() < 1e-10
    for simt in (False, True):
        got = c.gpu_decode(0, simt=simt)[0]
        print("errors (rel-L2, worst head, max-abs):", Hn.assert_attention_close(got, ref))


@pytest.mark.parametrize("simt", [False, True])
@pytest.mark.parametrize("splits", [1, 2, 7, 64])
def test_split_count_invariance(tiny, splits, simt):
    base = tiny.gpu_decode(0, num_splits=1, simt=simt)[0]
    got = tiny.gpu_decode(0, num_splits=splits, simt=simt)[0]
    assert np.abs(got - base).max() < (2e-5 if simt else 2e-4)
    ref, _ = tiny.oracle_attention(0)
    Hn.assert_attention_close(got, ref)


def test_export_import_roundtrip(layer7b_small):
    c = layer7b_small
    e = c.gpu_export(0)
    c2 = B.Cache(c.w.n_layers, c.w.batch, c.w.n_kv_heads, c.w.n_q_heads, c.cache.capacity)
    B.cache_import(c2, 0, e)
    torch.cuda.synchronize()
    npk_rec = (c.n // W) * B.RECORD_BYTES
    r1 = c.cache.records.view(c.w.batch * c.w.n_kv_heads, -1)[:, :npk_rec]
    r2 = c2.records.view(c.w.batch * c.w.n_kv_heads, -1)[:, :npk_rec]
    assert torch.equal(r1, r2)


def test_append_equals_bulk():
    """Appending tokens one by one gives bit-identical records, tails and lengths to bulk quantisation."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=2, n_layers=2)
    n0, n1 = 64 + 5, 64 + 5 + 70     # start mid-window, cross two window boundaries, end mid-window
    full = Hn.Case(w, n_tokens=n1, capacity=192)
    part = Hn.Case(w, n_tokens=n0, capacity=192)
    dev = part.cache.device
    for l in range(2):   # the same first n0 tokens as `full` (the generator's stream depends on the length)
        B.quantize_keys(part.cache, l, full.k[l][:, :, :n0].contiguous().to(dev), part.d_signs[l])
        B.quantize_values(part.cache, l, full.v[l][:, :, :n0].contiguous().to(dev),
                          full.mod_b[:, :n0].contiguous().to(dev), part.d_R[l])
    for i in range(n0, n1):
        k_new = torch.stack([full.k[l][:, :, i] for l in range(2)]).contiguous().to(dev)
        v_new = torch.stack([full.v[l][:, :, i] for l in range(2)]).contiguous().to(dev)
        m_new = full.mod_b[:, i].contiguous().to(dev)
        B.append(part.cache, 0, 2, k_new, v_new, m_new, part.d_signs, part.d_R)
    torch.cuda.synchronize()
    assert part.cache.device_status() == 0
    assert torch.equal(part.cache.seq_len, full.cache.seq_len)
    nrec = (n1 // W) * B.RECORD_BYTES
    U = 2 * w.batch * w.n_kv_heads
    assert torch.equal(part.cache.records.view(U, -1)[:, :nrec], full.cache.records.view(U, -1)[:, :nrec])
    nt = n1 % W
    assert torch.equal(part.cache.k_tail.view(U, W, D)[:, :nt], full.cache.k_tail.view(U, W, D)[:, :nt])
    assert torch.equal(part.cache.v_tail.view(U, W, D)[:, :nt], full.cache.v_tail.view(U, W, D)[:, :nt])
    assert torch.equal(part.cache.modality.view(w.batch, -1)[:, :n1], full.cache.modality.view(w.batch, -1)[:, :n1])
    # and decode over the appended cache (both layers in one call) matches the oracle
    got = part.gpu_decode(0, layer_count=2)
    for l in range(2):
        ref, _ = full.oracle_attention(l)
        Hn.assert_attention_close(got[l], ref)


def test_append_capacity_overflow_sets_status():
    w = WL.scaled(WL.WORKLOADS["tiny"])
    c = Hn.Case(w, n_tokens=64, capacity=64)
    k_new, v_new, m_new = WL.gen_new_token(w, 0, 0, device="cuda")
    before = c.cache.records.clone()
    B.append(c.cache, 0, 1, k_new[None].contiguous(), v_new[None].contiguous(), m_new, c.d_signs, c.d_R)
    torch.cuda.synchronize()
    assert c.cache.device_status() == B.ERR_CAPACITY
    assert c.cache.seq_len.cpu().tolist() == [64]
    assert torch.equal(before, c.cache.records)


def test_degenerate_inputs():
    w = WL.scaled(WL.WORKLOADS["tiny"])
    # empty cache -> zeros
    c = Hn.Case(w, n_tokens=0, capacity=64)
    assert (c.gpu_decode(0) == 0).all()
    # tail-only cache (n < 32) -> plain fp16 attention
    c = Hn.Case(w, n_tokens=21, capacity=64)
    ref, _ = c.oracle_attention(0)
    Hn.assert_attention_close(c.gpu_decode(0)[0], ref)
    # zero vectors and constant channels inside a window
    c = Hn.Case(w, n_tokens=64, capacity=64)
    k = c.k[0].clone(); v = c.v[0].clone()
    k[:, :, 3] = 0; v[:, :, 5] = 0; k[:, :, 32:64, :] = k[:, :, 32:33, :]
    c.k[0], c.v[0] = k, v
    B.quantize_keys(c.cache, 0, k.cuda(), c.d_signs[0]); B.quantize_values(c.cache, 0, v.cuda(), c.d_mod, c.d_R[0])
    kq, vq, _, _ = c.oracle_quantize(0)
    Hn.compare_cache(c, 0, c.gpu_export(0), kq, vq)
    ref, _ = c.oracle_attention(0)
    Hn.assert_attention_close(c.gpu_decode(0)[0], ref)


def test_per_head_rotations():
    """n_R = n_kv_heads: each KV head has its own set of three matrices."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], n_tokens=256)
    c = Hn.Case(w, n_tokens=256)
    Rh = torch.stack([WL.gen_rotations(w, 100 + h) for h in range(w.n_kv_heads)]).contiguous()   # [H,3,128,128]
    dRh = Rh.cuda()
    B.quantize_values(c.cache, 0, c.v[0].cuda(), c.d_mod, dRh)
    ws = torch.empty(B.decode_workspace_bytes(c.cache, 1, 0), dtype=torch.uint8, device="cuda")
    out = torch.empty(1, w.batch, w.n_q_heads, D, dtype=torch.float32, device="cuda")
    B.decode_attention(c.cache, 0, 1, c.d_q[0:1].contiguous(), c.d_signs[0:1].contiguous(), dRh, ws, out,
                       n_R=w.n_kv_heads)
    torch.cuda.synchronize()
    got = out[0].cpu().numpy().astype(np.float64)
    # oracle: one unit per head with its own rotation set
    U = w.n_kv_heads
    kb = Hn.u16(c.k[0]).reshape(U, 256, D); vb = Hn.u16(c.v[0]).reshape(U, 256, D)
    signs = np.tile(c.signs[0].numpy(), (U, 1))
    kq, vq, _ = O.quantize_batch(kb, vb, c.mod_b.numpy(), signs, Rh.numpy(), unit_rot=np.arange(U))
    q = Hn.u16(c.q[0]).reshape(U, w.group, D)
    ref, _ = O.attention(1, q, kq, vq, c.mod_b.numpy(), kb[:, 256:], vb[:, 256:], signs, Rh.numpy(), unit_rot=np.arange(U))
    Hn.assert_attention_close(got, ref.reshape(1, w.n_q_heads, D))


def _check_bulk_codes(c, layer, R_host):
    """Codes of the tensor-core value quantiser against the oracle: returns the number that differ (none may: the
    kernel recomputes every coordinate near a threshold with the reference arithmetic) after saying where."""
    kq, vq, _, vb = c.oracle_quantize(layer)
    e = {k: v.cpu() for k, v in c.gpu_export(layer).items()}
    U = c.w.batch * c.w.n_kv_heads
    cap, npk = c.cache.capacity, (c.n // W) * W
    assert (Hn.u16(e["v_norm"]).reshape(U, cap)[:, :npk] == vq["norm"]).all(), "value norms must be bit-identical"
    got = O.unpack_codes(e["v_codes"].numpy().reshape(U, cap, 32)[:, :npk])
    ref = O.unpack_codes(vq["codes"])
    bad = np.argwhere(got != ref)
    _, T = O.codebook()
    thr = np.array([-T, 0.0, T], dtype=np.float64)
    unit_seq = np.repeat(np.arange(c.w.batch), c.w.n_kv_heads)
    for (u, i, ch) in bad:
        m = c.mod_b.numpy()[unit_seq[u], i]
        _, z = O.value_rotate(vb[u, i], R_host[m])
        print("value code differs:", (u, i, ch), int(got[u, i, ch]), int(ref[u, i, ch]), "distance to threshold",
              np.abs(float(z[ch]) - thr).min())
    return len(bad), ref.size


def test_bulk_value_quantiser_on_tensor_cores():
    # several 128-token tiles, mixed-modality tiles, a partial last tile (2048 + 64 + 19 tokens)
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=2)
    c = Hn.Case(w, n_tokens=2048 + 64 + 19)
    dev = c.cache.device
    B.quantize_values(c.cache, 0, c.v[0].to(dev), c.d_mod, c.d_R[0], bulk=True)
    torch.cuda.synchronize()
    assert c.cache.device_status() == 0
    n_bad, n_all = _check_bulk_codes(c, 0, c.R[0].numpy())
    assert n_bad == 0, f"{n_bad} of {n_all} tensor-core value codes differ from the exact chain"
    # decode over the bulk-built cache matches the oracle
    ref, _ = c.oracle_attention(0)
    Hn.assert_attention_close(c.gpu_decode(0)[0], ref)
    # raw tail and modality as in the exact path
    U = w.batch * w.n_kv_heads
    assert (Hn.u16(c.cache.v_tail).reshape(U, W, D)[:, :19] == Hn.u16(c.v[0]).reshape(U, c.n, D)[:, 2048 + 64:]).all()
    # a signed permutation is rotated exactly by any arithmetic: codes must then be identical
    rng = np.random.default_rng(5)
    P = np.zeros((3, D, D), np.float32)
    for m in range(3):
        P[m, np.arange(D), rng.permutation(D)] = np.where(rng.random(D) < 0.5, -1.0, 1.0)
    c.R[0] = torch.from_numpy(P)
    dP = torch.from_numpy(P)[None].contiguous().to(dev)
    B.quantize_values(c.cache, 0, c.v[0].to(dev), c.d_mod, dP, bulk=True)
    torch.cuda.synchronize()
    n_bad, _ = _check_bulk_codes(c, 0, P)
    assert n_bad == 0
