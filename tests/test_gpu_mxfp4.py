"""GPU parity of the MXFP4-metadata cache format (the paper's default (m, s) storage, 2.258 bits per
element): stored bytes, decoded pairs, codes and norms bit for bit against the oracle; decode
attention within the tolerance of the fp16-metadata path."""
import numpy as np
import pytest
import torch

from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL
from tests import harness as Hn

pytestmark = pytest.mark.gpu
D, W = 128, 32
MX = B.META_MXFP4


@pytest.fixture(scope="module")
def tiny_mx():
    return Hn.Case(WL.WORKLOADS["tiny"], meta_format=MX)


@pytest.fixture(scope="module")
def ragged_mx():
    # odd number of whole windows (65) so that the last 4624-byte window pair is half used
    return Hn.Case(WL.scaled(WL.WORKLOADS["layer7b"], batch=2), n_tokens=65 * W + 19, meta_format=MX)


def test_record_bytes():
    sizes = B.cache_sizes(1, 1, 1, 1, 64 * W, meta_format=MX)
    assert sizes[0] == 64 * 2312            # 72.25 bytes per token and KV head
    assert B.cache_sizes(1, 1, 1, 1, 3 * W, meta_format=MX)[0] == 2 * 4624   # windows are stored in pairs
    assert B.cache_sizes(1, 1, 1, 1, 64 * W)[0] == 64 * 2688


def test_quantize_bit_exact(tiny_mx, ragged_mx):
    for c in (tiny_mx, ragged_mx):
        kq, vq, _, _ = c.oracle_quantize(0)
        assert "mx" in kq
        Hn.compare_cache(c, 0, c.gpu_export(0), kq, vq)
        assert c.cache.device_status() == 0


@pytest.mark.parametrize("simt", [False, True])
def test_decode_matches_oracle(tiny_mx, ragged_mx, simt):
    for c in (tiny_mx, ragged_mx):
        ref, _ = c.oracle_attention(0)
        got = c.gpu_decode(0, simt=simt)[0]
        print("errors (rel-L2, worst head, max-abs):", Hn.assert_attention_close(got, ref))


@pytest.mark.parametrize("splits", [1, 3, 16])
def test_split_count_invariance(ragged_mx, splits):
    ref, _ = ragged_mx.oracle_attention(0)
    Hn.assert_attention_close(ragged_mx.gpu_decode(0, num_splits=splits)[0], ref)


def test_append_equals_bulk():
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=2)
    n0, n1 = 3 * W + 5, 5 * W + 7
    full = Hn.Case(w, n_tokens=n1, meta_format=MX)
    part = B.Cache(w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, full.cache.capacity, meta_format=MX)
    k, v = full.k[0].cuda(), full.v[0].cuda()
    B.quantize_keys(part, 0, k[:, :, :n0].contiguous(), full.d_signs[0])
    B.quantize_values(part, 0, v[:, :, :n0].contiguous(), full.d_mod[:, :n0].contiguous(), full.d_R[0])
    for i in range(n0, n1):
        B.append(part, 0, 1, k[:, :, i].contiguous().unsqueeze(0), v[:, :, i].contiguous().unsqueeze(0),
                 full.d_mod[:, i].contiguous(), full.d_signs[0:1], full.d_R[0:1])
    torch.cuda.synchronize()
    assert part.device_status() == 0
    a, b = B.cache_export(part, 0), B.cache_export(full.cache, 0)
    nw = n1 // W
    for key in a:
        x, y = a[key].cpu(), b[key].cpu()
        lim = nw if key in ("k_meta", "k_mx") else nw * W
        assert torch.equal(x[:, :, :lim], y[:, :, :lim]), key
    U, nt = w.batch * w.n_kv_heads, n1 % W      # rows past the live tail are stale in the appended cache
    assert torch.equal(part.k_tail.view(U, W, D)[:, :nt], full.cache.k_tail.view(U, W, D)[:, :nt])
    assert torch.equal(part.v_tail.view(U, W, D)[:, :nt], full.cache.v_tail.view(U, W, D)[:, :nt])
    assert part.seq_len.cpu().tolist() == full.cache.seq_len.cpu().tolist()


def test_bulk_value_quantiser_writes_the_same_bodies():
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=2)
    a = Hn.Case(w, n_tokens=8 * W, meta_format=MX)
    b = Hn.Case(w, n_tokens=8 * W, meta_format=MX, bulk_values=True)
    ea, eb = a.gpu_export(0), b.gpu_export(0)
    assert torch.equal(ea["v_norm"], eb["v_norm"]) and torch.equal(ea["k_mx"], eb["k_mx"])
    # the tensor-core rotation may move a value across a codebook threshold it sits on
    assert (ea["v_codes"] != eb["v_codes"]).sum().item() <= 4


def test_import_is_refused_and_formats_agree_on_bodies():
    w = WL.WORKLOADS["tiny"]
    mx = Hn.Case(w, meta_format=MX)
    fp = Hn.Case(w)
    e = B.cache_export(mx.cache, 0)
    with pytest.raises(B.OkqError) as ei:
        B.cache_import(mx.cache, 0, {k: v for k, v in e.items() if k != "k_mx"})
    assert ei.value.status == B.ERR_UNSUPPORTED
    f = B.cache_export(fp.cache, 0)
    for key in ("k_norm", "v_norm", "v_codes"):    # independent of the metadata format
        assert torch.equal(e[key], f[key]), key
    # the decoded MX pairs are the fp16 pairs rounded to one mantissa bit: within a quarter of their magnitude,
    # except near zero of a block (absolute step 2^k / 2) and in the saturating top quarter of a block
    me, mf = e["k_meta"].float().cpu(), f["k_meta"].float().cpu()
    nw = 2048 // W
    me, mf = me[:, :, :nw], mf[:, :, :nw]
    blk_max = mf[..., 0].abs().reshape(*mf.shape[:3], 4, 32).amax(-1, keepdim=True).expand(-1, -1, -1, -1, 32).reshape(mf[..., 0].shape)
    assert ((me[..., 0] - mf[..., 0]).abs() <= torch.maximum(mf[..., 0].abs() / 4, blk_max / 16) + 1e-6).all()
