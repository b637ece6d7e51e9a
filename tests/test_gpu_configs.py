"""GPU parity on the benchmark's other shapes and at the full size the benchmark times.

  * 30B-A3B shape (GQA group 8, video 400 / audio 100 chunks), reduced layers and context;
  * long-context decode (batch 1, many CTAs per (sequence, head));
  * long single-modality ranges per warp pair, and thousands of two-window units in one launch;
  * the full 7B decode step (28 layers x batch 8 x 16384 tokens, one append + one decode call
    over all layers, inputs drawn on the GPU exactly as bench.py does), checked on sampled
    (layer, sequence) pairs the oracle can afford, plus properties that hold at any size.
"""
import numpy as np
import pytest
import torch

from oracle import okq_oracle as O
from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL
from tests import harness as Hn

pytestmark = pytest.mark.gpu
D, W = 128, 32


def test_group8_30b_shape():
    w = WL.scaled(WL.WORKLOADS["step30b"], n_layers=2, batch=2, n_tokens=4096 + 7)
    c = Hn.Case(w)
    for l in range(2):
        kq, vq, _, _ = c.oracle_quantize(l)
        Hn.compare_cache(c, l, c.gpu_export(l), kq, vq)
    got = c.gpu_decode(0, layer_count=2)
    for l in range(2):
        ref, _ = c.oracle_attention(l)
        print("30B shape layer", l, Hn.assert_attention_close(got[l], ref))
    simt = c.gpu_decode(0, layer_count=2, simt=True)
    assert np.abs(simt - got).max() < 1e-3


def test_long_context_batch1():
    w = WL.scaled(WL.WORKLOADS["long7b"], n_layers=1, n_tokens=32768 + 31)
    c = Hn.Case(w)
    ref, _ = c.oracle_attention(0)
    got = c.gpu_decode(0)[0]                 # 148 CTAs over 4 (sequence, head) units: 37 partials each
    print("long context", Hn.assert_attention_close(got, ref))
    got4 = c.gpu_decode(0, num_splits=3)[0]
    Hn.assert_attention_close(got4, ref)


def test_one_modality_long_ranges():
    """One warp pair covers 256 windows of a single modality (one CTA per (sequence, head), no modality change
    that would move the register sums out): the value sums must not drift with the length of the range.  The
    tensor cores accumulate without rounding to nearest, so a long chain into one register is biased; the
    kernel bounds the chain, and this case fails (worst head above the tolerance) if it does not."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], n_tokens=65536 + 3)
    c = Hn.Case(w, modality=torch.zeros(w.n_tokens, dtype=torch.uint8))
    ref, _ = c.oracle_attention(0)
    for splits in (1, 0):
        got = c.gpu_decode(0, num_splits=splits)[0]
        errs = Hn.assert_attention_close(got, ref)
        assert errs[1] < 6e-4, errs      # worst head: well inside the 1e-3 tolerance
        print("one modality, splits", splits, errs)


@pytest.mark.parametrize("meta_format", [B.META_FP16, B.META_MXFP4])
def test_middle_sized_grid(meta_format):
    """64 (head, four-sequence group, layer) blocks: fewer than SMs but too many for four column slices each, the
    case in which the combine kernel runs one sequence per block over all columns."""
    w = WL.scaled(WL.WORKLOADS["step7b"], n_layers=8, n_tokens=1024 + 7)
    c = Hn.Case(w, meta_format=meta_format)
    got = c.gpu_decode(0, layer_count=w.n_layers)
    for l in (0, 3, 7):
        ref, _ = c.oracle_attention(l)
        Hn.assert_attention_close(got[l], ref)


def test_one_head_over_every_cta():
    """A single (sequence, head) unit of 129 windows: every CTA of the split-K kernel holds one window of it, so the
    combine kernel merges 129 partials for one head group, more than its table of precomputed factors holds."""
    w = WL.scaled(WL.WORKLOADS["tiny"], n_tokens=4128 + 5, n_chunks=0)
    c = Hn.Case(w)
    ref, _ = c.oracle_attention(0)
    got = c.gpu_decode(0)[0]
    print("one head over every CTA", Hn.assert_attention_close(got, ref))


def test_decode_is_deterministic():
    """No atomics and a fixed partition: two calls on the same cache give bit-identical outputs (both grids)."""
    w = WL.scaled(WL.WORKLOADS["step7b"], n_layers=2, batch=3, n_tokens=2048 + 17)
    c = Hn.Case(w)
    for splits in (0, 2):
        a = c.gpu_decode(0, layer_count=2, num_splits=splits)
        b = c.gpu_decode(0, layer_count=2, num_splits=splits)
        assert np.array_equal(a, b)


def test_many_short_units_per_cta():
    """8192 (sequence, head) units of two windows each in one launch: every warp pair crosses several unit
    boundaries and every CTA merges ~55 units, more than one batch of its end-of-launch merge."""
    w = WL.Workload("short", 5, 8, 128, 16, 8, 64 + 5, 16, 20, 12, 0)
    c = Hn.Case(w)
    got = c.gpu_decode(0, layer_count=w.n_layers)
    for l in range(w.n_layers):
        ref, _ = c.oracle_attention(l)
        Hn.assert_attention_close(got[l], ref)
    assert c.cache.device_status() == 0


@pytest.mark.parametrize("meta_format", [B.META_FP16, B.META_MXFP4])
def test_full_7b_step_sampled(meta_format):
    w = WL.WORKLOADS["step7b"]
    dev = torch.device("cuda")
    L, Bn, H, Hq, N = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.n_tokens
    cache = B.Cache(L, Bn, H, Hq, N + 64, device=dev, meta_format=meta_format)
    mod_cpu = WL.modality_layout(w)
    mod = mod_cpu.unsqueeze(0).repeat(Bn, 1).contiguous().to(dev)
    signs = torch.stack([WL.gen_signs(w, l) for l in range(L)])
    R = torch.stack([WL.gen_rotations(w, l) for l in range(L)])
    d_signs, d_R = signs.to(dev), R.unsqueeze(1).contiguous().to(dev)
    samples = [(0, 0), (13, 5), (27, 7)]
    kept = {}
    for l in range(L):
        k, v = WL.gen_kv(w, l, device=dev)
        B.quantize_keys(cache, l, k, d_signs[l])
        B.quantize_values(cache, l, v, mod, d_R[l])
        for (sl, sb) in samples:
            if sl == l:
                kept[(sl, sb)] = (k[sb].cpu(), v[sb].cpu())
        del k, v
    q = torch.stack([WL.gen_queries(w, l) for l in range(L)])
    d_q = q.to(dev)
    k_new, v_new, m_new = WL.gen_new_token(w, 0, 0, device=dev)
    kn = k_new.unsqueeze(0).expand(L, -1, -1, -1).contiguous()
    vn = v_new.unsqueeze(0).expand(L, -1, -1, -1).contiguous()
    B.append(cache, 0, L, kn, vn, m_new, d_signs, d_R)
    ws = torch.empty(B.decode_workspace_bytes(cache, L, 0), dtype=torch.uint8, device=dev)
    out = torch.full((L, Bn, Hq, D), float("nan"), dtype=torch.float32, device=dev)
    B.decode_attention(cache, 0, L, d_q, d_signs, d_R, ws, out)
    torch.cuda.synchronize()
    assert cache.device_status() == 0
    assert (cache.seq_len == N + 1).all()
    o = out.cpu().numpy().astype(np.float64)
    # properties at any size: finite, and an attention output is a convex combination of value
    # vectors, so its norm cannot exceed the largest value norm (reconstruction adds at most ~35 %)
    assert np.isfinite(o).all()
    assert np.linalg.norm(o, axis=-1).max() < 6.0
    # sampled (layer, sequence) pairs against the oracle: packed cache bit for bit, attention within tolerance
    for (sl, sb) in samples:
        kc, vc = kept[(sl, sb)]
        kb = Hn.u16(kc).reshape(H, N, D); vb = Hn.u16(vc).reshape(H, N, D)
        kq, vq, _ = O.quantize_batch(kb, vb, mod_cpu.numpy(), signs[sl].numpy(), R[sl].numpy(), meta_format=meta_format)
        e = B.cache_export(cache, sl)
        torch.cuda.synchronize()
        cap = cache.capacity
        assert (e["k_codes"][sb].cpu().numpy()[:, :N] == kq["codes"]).all()
        assert (Hn.u16(e["k_norm"][sb])[:, :N] == kq["norm"]).all()
        assert (Hn.u16(e["k_meta"][sb])[:, :N // W] == kq["meta"]).all()
        if meta_format == B.META_MXFP4:
            assert (e["k_mx"][sb].cpu().numpy()[:, :N // W] == kq["mx"]).all()
        assert (e["v_codes"][sb].cpu().numpy()[:, :N] == vq["codes"]).all()
        assert (Hn.u16(e["v_norm"][sb])[:, :N] == vq["norm"]).all()
        del e
        qs = Hn.u16(q[sl, sb]).reshape(H, w.group, D)
        kt = np.broadcast_to(Hn.u16(k_new[sb].cpu())[:, None, :], (H, 1, D))
        vt = np.broadcast_to(Hn.u16(v_new[sb].cpu())[:, None, :], (H, 1, D))
        modrow = np.concatenate([mod_cpu.numpy(), np.zeros(1, np.uint8)])
        ref, _ = O.attention(1, qs, kq, vq, modrow, kt, vt, signs[sl].numpy(), R[sl].numpy())
        errs = Hn.assert_attention_close(o[sl, sb], ref.reshape(Hq, D))
        print(f"full step7b (meta format {meta_format}) layer {sl} seq {sb}: rel-L2 {errs[0]:.2e} worst head {errs[1]:.2e} max-abs {errs[2]:.2e}")


@pytest.mark.parametrize("meta_format", [B.META_FP16, B.META_MXFP4])
def test_every_window_holds_all_three_modalities(meta_format):
    """Worst case for the per-modality bookkeeping: modality ids drawn per token, so every 32-token window
    (and every 128-token tile of the bulk value quantiser) mixes text, audio and video; a few ids > 2, which
    count as text."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=2)
    n = 1024 + 13
    g = torch.Generator().manual_seed(99)
    mod = torch.randint(0, 3, (n,), generator=g, dtype=torch.uint8)
    mod[::97] = 7
    c = Hn.Case(w, n_tokens=n, meta_format=meta_format, modality=mod)
    kq, vq, _, _ = c.oracle_quantize(0)
    Hn.compare_cache(c, 0, c.gpu_export(0), kq, vq)
    assert (c.cache.modality.view(w.batch, -1)[:, :n].cpu() == torch.where(mod > 2, torch.zeros_like(mod), mod)).all()
    ref, _ = c.oracle_attention(0)
    print("mixed windows:", Hn.assert_attention_close(c.gpu_decode(0)[0], ref))
    Hn.assert_attention_close(c.gpu_decode(0, simt=True)[0], ref)
    # the tensor-core value quantiser on the same input: two jobs per tile (three modalities, two accumulators)
    b = Hn.Case(w, n_tokens=n, meta_format=meta_format, modality=mod, bulk_values=True)
    ea, eb = c.gpu_export(0), b.gpu_export(0)
    assert b.cache.device_status() == 0
    assert torch.equal(ea["v_norm"], eb["v_norm"])
    assert torch.equal(ea["v_codes"], eb["v_codes"])               # the bulk path fixes up coordinates near a threshold
    Hn.assert_attention_close(b.gpu_decode(0)[0], ref)


def test_ragged_batch_lengths():
    """Sequences of different lengths in one decode call (lengths set per sequence, tails filled to match):
    the persistent kernel's partition follows the per-sequence window counts."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=4, n_layers=2, n_tokens=1500)
    c = Hn.Case(w, capacity=1536)
    dev = c.cache.device
    lengths = np.array([[1500, 40, 700, 0], [33, 1499, 31, 1024]])        # [layer][sequence]
    U = w.batch * w.n_kv_heads
    kt = c.cache.k_tail.view(2, w.batch, w.n_kv_heads, W, D)
    vt = c.cache.v_tail.view(2, w.batch, w.n_kv_heads, W, D)
    for l in range(2):
        for b in range(w.batch):
            n = int(lengths[l, b]); npk = (n // W) * W
            if n > npk:
                kt[l, b, :, : n - npk] = c.k[l][b, :, npk:n].to(dev)
                vt[l, b, :, : n - npk] = c.v[l][b, :, npk:n].to(dev)
    c.cache.seq_len.copy_(torch.from_numpy(lengths.reshape(-1).astype(np.int32)).to(dev))
    got = c.gpu_decode(0, layer_count=2)
    got_simt = c.gpu_decode(0, layer_count=2, simt=True)
    for l in range(2):
        for b in range(w.batch):
            n = int(lengths[l, b])
            if n == 0:
                assert (got[l, b] == 0).all() and (got_simt[l, b] == 0).all()
                continue
            kb = Hn.u16(c.k[l][b, :, :n]); vb = Hn.u16(c.v[l][b, :, :n])
            mod = c.mod_b[b, :n].numpy()
            kq, vq, _ = O.quantize_batch(kb, vb, mod, c.signs[l].numpy(), c.R[l].numpy())
            npk = (n // W) * W
            q = Hn.u16(c.q[l, b]).reshape(w.n_kv_heads, w.group, D)
            ref, _ = O.attention(1, q, kq, vq, mod, kb[:, npk:], vb[:, npk:], c.signs[l].numpy(), c.R[l].numpy())
            ref = ref.reshape(w.n_q_heads, D)
            Hn.assert_attention_close(got[l, b], ref)
            Hn.assert_attention_close(got_simt[l, b], ref)


@pytest.mark.parametrize("n_q,n_kv", [(4, 4), (8, 2), (6, 1)])
def test_other_gqa_groups(n_q, n_kv):
    """GQA groups 1, 4 and 6 (the kernels pad the group to 8 heads)."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], n_q_heads=n_q, n_kv_heads=n_kv, batch=2, n_tokens=300 + 11)
    c = Hn.Case(w)
    ref, _ = c.oracle_attention(0)
    Hn.assert_attention_close(c.gpu_decode(0)[0], ref)
    Hn.assert_attention_close(c.gpu_decode(0, simt=True)[0], ref)


def test_layer_offset_and_many_sequences():
    """A call on layers [1, 3) of a 3-layer cache with more (layer, sequence) pairs than one launch
    covers (the library then launches layer by layer)."""
    w = WL.scaled(WL.WORKLOADS["tiny"], n_layers=3, batch=600, n_tokens=40)
    c = Hn.Case(w, capacity=64)
    got = c.gpu_decode(1, layer_count=2)
    for i, l in enumerate((1, 2)):
        ref, _ = c.oracle_attention(l)
        Hn.assert_attention_close(got[i], ref)
