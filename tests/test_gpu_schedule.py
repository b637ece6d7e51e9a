"""GPU parity of the captioning schedule (keys packed every 128 tokens, values behind a 128-token fp16
window): cache state after bulk prefill and after token-by-token append, and decode attention against
the oracle's definition, at lengths around every boundary of the schedule."""
import numpy as np
import pytest
import torch

from oracle import okq_oracle as O
from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL
from tests import harness as Hn

pytestmark = pytest.mark.gpu
D, W = 128, 32
CAP = B.SCHEDULE_CAPTION


def _inputs(n, batch=2, seed_layer=0):
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=batch)
    k, v = WL.gen_kv(w, seed_layer, n_tokens=n)
    mod = WL.modality_layout(w, n)
    signs = WL.gen_signs(w, seed_layer)
    R = WL.gen_rotations(w, seed_layer)
    q = WL.gen_queries(w, seed_layer)
    return w, k, v, mod, signs, R, q


def _decode(cache, w, q, signs, R):
    ws = torch.empty(max(16, B.decode_workspace_bytes(cache, 1, 0)), dtype=torch.uint8, device="cuda")
    out = torch.full((1, w.batch, w.n_q_heads, D), float("nan"), dtype=torch.float32, device="cuda")
    B.decode_attention(cache, 0, 1, q.cuda()[None], signs.cuda()[None], R.cuda()[None, None], ws, out)
    torch.cuda.synchronize()
    return out[0].cpu().numpy().astype(np.float64)


def _oracle(w, k, v, mod, signs, R, q, n, meta_format):
    kp, vp = O.packed_counts(n, 1)
    ref = np.zeros((w.batch, w.n_q_heads, D))
    G = w.group
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            kb = Hn.u16(k[b, h, :n]); vb = Hn.u16(v[b, h, :n])
            kq, vq, _ = O.quantize_batch(kb[None], vb[None], mod.numpy()[:n], signs.numpy(), R.numpy(), meta_format=meta_format)
            kq1 = {a: x[0] for a, x in kq.items()}; vq1 = {a: x[0] for a, x in vq.items()}
            ref[b, h * G:(h + 1) * G] = O.attention_scheduled(Hn.u16(q[b, h * G:(h + 1) * G]), kq1, vq1, mod.numpy(), kb, vb,
                                                              signs.numpy(), R.numpy(), kp, vp)
    return ref


def test_buffer_sizes():
    s = B.cache_sizes(2, 3, 4, 28, 1024, schedule=CAP)
    units = 2 * 3 * 4
    assert s[2] == units * 128 * D * 2 and s[3] == units * 160 * D * 2          # raw key / value slots
    assert s[0] == B.cache_sizes(2, 3, 4, 28, 1024)[0]                            # the records do not change


@pytest.mark.parametrize("n", [5, 127, 128, 159, 160, 255, 256, 300, 1024 + 77])
@pytest.mark.parametrize("meta_format", [B.META_FP16, B.META_MXFP4])
def test_bulk_prefill_then_decode(n, meta_format):
    w, k, v, mod, signs, R, q = _inputs(n)
    cache = B.Cache(1, w.batch, w.n_kv_heads, w.n_q_heads, ((n + 31) // 32 + 2) * 32, meta_format=meta_format, schedule=CAP)
    modb = mod[None].repeat(w.batch, 1).contiguous().cuda()
    B.quantize_keys(cache, 0, k.cuda(), signs.cuda())
    B.quantize_values(cache, 0, v.cuda(), modb, R.cuda()[None], bulk=(n % 2 == 0))   # both value quantisers
    torch.cuda.synchronize()
    assert cache.device_status() == 0 and cache.seq_len.cpu().tolist() == [n] * w.batch
    got = _decode(cache, w, q, signs, R)
    ref = _oracle(w, k, v, mod, signs, R, q, n, meta_format)
    print(f"n={n} meta {meta_format}:", Hn.assert_attention_close(got, ref))
    # the cross-check kernels know the window schedule only
    ws = torch.empty(max(16, B.decode_workspace_bytes(cache, 1, 0)), dtype=torch.uint8, device="cuda")
    out = torch.empty(1, w.batch, w.n_q_heads, D, dtype=torch.float32, device="cuda")
    with pytest.raises(B.OkqError) as ei:
        B.decode_attention(cache, 0, 1, q.cuda()[None], signs.cuda()[None], R.cuda()[None, None], ws, out, simt=True)
    assert ei.value.status == B.ERR_UNSUPPORTED


def test_append_equals_bulk_and_decode_at_every_step():
    """Token-by-token append under the captioning schedule: records, raw slots and lengths equal those of a bulk
    prefill of the same tokens, and the decode output matches the oracle across the schedule's boundaries."""
    n0, n1 = 100, 420
    w, k, v, mod, signs, R, q = _inputs(n1)
    cap = 448
    part = B.Cache(1, w.batch, w.n_kv_heads, w.n_q_heads, cap, schedule=CAP)
    modb = mod[None].repeat(w.batch, 1).contiguous().cuda()
    kd, vd = k.cuda(), v.cuda()
    B.quantize_keys(part, 0, kd[:, :, :n0].contiguous(), signs.cuda())
    B.quantize_values(part, 0, vd[:, :, :n0].contiguous(), modb[:, :n0].contiguous(), R.cuda()[None])
    check_at = {127, 128, 129, 159, 160, 161, 255, 256, 288, 319, 320, 384, n1}
    for i in range(n0, n1):
        B.append(part, 0, 1, kd[:, :, i].contiguous()[None], vd[:, :, i].contiguous()[None], modb[:, i].contiguous(),
                 signs.cuda()[None], R.cuda()[None, None])
        n = i + 1
        if n in check_at:
            torch.cuda.synchronize()
            assert part.device_status() == 0 and part.seq_len.cpu().tolist() == [n] * w.batch
            full = B.Cache(1, w.batch, w.n_kv_heads, w.n_q_heads, cap, schedule=CAP)
            B.quantize_keys(full, 0, kd[:, :, :n].contiguous(), signs.cuda())
            B.quantize_values(full, 0, vd[:, :, :n].contiguous(), modb[:, :n].contiguous(), R.cuda()[None])
            kp, vp = O.packed_counts(n, 1)
            ea, eb = B.cache_export(part, 0), B.cache_export(full, 0)
            for key, lim in (("k_codes", kp), ("k_norm", kp), ("k_meta", kp // W), ("v_codes", vp), ("v_norm", vp)):
                assert torch.equal(ea[key][:, :, :lim], eb[key][:, :, :lim]), (n, key)
            U = w.batch * w.n_kv_heads
            kt_a, kt_b = part.k_tail.view(U, 128, D), full.k_tail.view(U, 128, D)
            vt_a, vt_b = part.v_tail.view(U, 160, D), full.v_tail.view(U, 160, D)
            ks = torch.tensor([t % 128 for t in range(kp, n)], dtype=torch.long, device="cuda")
            vs = torch.tensor([t % 160 for t in range(vp, n)], dtype=torch.long, device="cuda")
            assert torch.equal(kt_a[:, ks], kt_b[:, ks]) and torch.equal(vt_a[:, vs], vt_b[:, vs]), n
            assert torch.equal(kt_a[:, ks].cpu(), k[:, :, kp:n].reshape(U, n - kp, D))
            got = _decode(part, w, q, signs, R)
            ref = _oracle(w, k, v, mod, signs, R, q, n, B.META_FP16)
            Hn.assert_attention_close(got, ref)


@pytest.mark.parametrize("schedule", [B.SCHEDULE_WINDOW, CAP])
def test_full_size_batched_call_equals_per_layer_calls(schedule):
    """The 28-layer call runs the combine kernel in its four-sequences-per-block configuration, a single-layer call
    in the one-sequence configuration (which the small cases above reach and check against the oracle).  Both must
    give the same attention output up to the rounding of a different split of the windows; repeated a few steps so
    that a timing-dependent fault between the sequence groups of a block would show (non-finite or far-off values)."""
    w = WL.WORKLOADS["step7b"]
    dev = torch.device("cuda")
    L, Bn, H, Hq, N = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.n_tokens
    cache = B.Cache(L, Bn, H, Hq, N + 64, device=dev, schedule=schedule)
    mod = WL.modality_layout(w).unsqueeze(0).repeat(Bn, 1).contiguous().to(dev)
    signs = torch.stack([WL.gen_signs(w, l) for l in range(L)]).to(dev)
    R = torch.stack([WL.gen_rotations(w, l) for l in range(L)]).unsqueeze(1).contiguous().to(dev)
    for l in range(L):
        k, v = WL.gen_kv(w, l, device=dev)
        B.quantize_keys(cache, l, k, signs[l])
        B.quantize_values(cache, l, v, mod, R[l], bulk=True)
        del k, v
    q = torch.stack([WL.gen_queries(w, l) for l in range(L)]).to(dev)
    ws = torch.empty(B.decode_workspace_bytes(cache, L, 0), dtype=torch.uint8, device=dev)
    for s in range(6):
        kn, vn, mn = WL.gen_new_token(w, 0, s, device=dev)
        kn = kn.unsqueeze(0).expand(L, -1, -1, -1).contiguous()
        vn = vn.unsqueeze(0).expand(L, -1, -1, -1).contiguous()
        B.append(cache, 0, L, kn, vn, mn, signs, R)
        a = torch.full((L, Bn, Hq, D), float("nan"), dtype=torch.float32, device=dev)
        b = torch.full_like(a, float("nan"))
        B.decode_attention(cache, 0, L, q, signs, R, ws, a)
        for l in range(L):
            B.decode_attention(cache, l, 1, q[l:l + 1], signs[l:l + 1], R[l:l + 1], ws, b[l:l + 1])
        torch.cuda.synchronize()
        assert torch.isfinite(a).all() and torch.isfinite(b).all(), s
        assert (a - b).abs().max().item() < 2e-3, (s, (a - b).abs().max().item())
    assert cache.device_status() == 0


def _check_sampled(cache, w, samples, kept, q, signs, R, mod_row, n, out, meta_format):
    """Sampled (layer, sequence) pairs of a caption-schedule cache of `n` tokens per sequence against the oracle:
    packed records bit for bit up to the schedule's packed counts, attention output within the tolerance."""
    H, G = w.n_kv_heads, w.group
    kp, vp = O.packed_counts(n, 1)
    for (sl, sb) in samples:
        kc, vc = kept[(sl, sb)]                                  # [H, n, 128] fp16, host
        kb, vb = Hn.u16(kc), Hn.u16(vc)
        kq, vq, _ = O.quantize_batch(kb, vb, mod_row, signs[sl].numpy(), R[sl].numpy(), meta_format=meta_format)
        e = B.cache_export(cache, sl)
        torch.cuda.synchronize()
        assert (e["k_codes"][sb].cpu().numpy()[:, :kp] == kq["codes"][:, :kp]).all()
        assert (Hn.u16(e["k_norm"][sb])[:, :kp] == kq["norm"][:, :kp]).all()
        assert (Hn.u16(e["k_meta"][sb])[:, :kp // W] == kq["meta"][:, :kp // W]).all()
        assert (e["v_codes"][sb].cpu().numpy()[:, :vp] == vq["codes"][:, :vp]).all()
        assert (Hn.u16(e["v_norm"][sb])[:, :vp] == vq["norm"][:, :vp]).all()
        del e
        ref = np.zeros((w.n_q_heads, D))
        for h in range(H):
            kq1 = {a: x[h] for a, x in kq.items()}; vq1 = {a: x[h] for a, x in vq.items()}
            ref[h * G:(h + 1) * G] = O.attention_scheduled(Hn.u16(q[sl, sb, h * G:(h + 1) * G]), kq1, vq1, mod_row, kb[h], vb[h],
                                                           signs[sl].numpy(), R[sl].numpy(), kp, vp)
        errs = Hn.assert_attention_close(out[sl, sb], ref)
        print(f"caption n={n} meta {meta_format} layer {sl} seq {sb}: rel-L2 {errs[0]:.2e} worst head {errs[1]:.2e} max-abs {errs[2]:.2e}")


@pytest.mark.parametrize("meta_format", [B.META_FP16, B.META_MXFP4])
def test_middle_sized_grid_caption(meta_format):
    """Captioning schedule with 64 (head, four-sequence group, layer) combine blocks: fewer than SMs but too many for
    four column slices each, so the combine kernel runs one sequence per block over all output columns; every
    sequence holds packed keys whose values are still raw, raw keys and raw values.  Against the oracle."""
    w = WL.scaled(WL.WORKLOADS["step7b"], n_layers=8, n_tokens=1024 + 77)
    n, L, dev = w.n_tokens, w.n_layers, torch.device("cuda")
    cache = B.Cache(L, w.batch, w.n_kv_heads, w.n_q_heads, ((n + 31) // 32 + 2) * 32, device=dev, meta_format=meta_format, schedule=CAP)
    mod_cpu = WL.modality_layout(w)
    mod = mod_cpu.unsqueeze(0).repeat(w.batch, 1).contiguous().to(dev)
    signs = torch.stack([WL.gen_signs(w, l) for l in range(L)])
    R = torch.stack([WL.gen_rotations(w, l) for l in range(L)])
    q = torch.stack([WL.gen_queries(w, l) for l in range(L)])
    d_signs, d_R = signs.to(dev), R.unsqueeze(1).contiguous().to(dev)
    samples = [(0, 0), (3, 5), (7, 2), (7, 7)]
    kept = {}
    for l in range(L):
        k, v = WL.gen_kv(w, l)
        B.quantize_keys(cache, l, k.to(dev), d_signs[l])
        B.quantize_values(cache, l, v.to(dev), mod, d_R[l], bulk=(l % 2 == 0))
        for (sl, sb) in samples:
            if sl == l:
                kept[(sl, sb)] = (k[sb], v[sb])
    ws = torch.empty(B.decode_workspace_bytes(cache, L, 0), dtype=torch.uint8, device=dev)
    out = torch.full((L, w.batch, w.n_q_heads, D), float("nan"), dtype=torch.float32, device=dev)
    B.decode_attention(cache, 0, L, q.to(dev), d_signs, d_R, ws, out)
    torch.cuda.synchronize()
    assert cache.device_status() == 0
    o = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(o).all()
    _check_sampled(cache, w, samples, kept, q, signs, R, mod_cpu.numpy(), n, o, meta_format)


@pytest.mark.parametrize("meta_format", [B.META_FP16, B.META_MXFP4])
def test_full_7b_step_caption_sampled(meta_format):
    """The full 7B decode step under the captioning schedule (28 layers x batch 8, one append call and one decode call
    over all layers: the combine kernel's four-sequences-per-block configuration), after 45 appended tokens that cross
    a 32-token boundary (a value window leaves the fp16 window) and a 128-token boundary (four key windows are
    packed); sampled (layer, sequence) pairs against the oracle."""
    w0 = WL.WORKLOADS["step7b"]
    n0, n_app = w0.n_tokens - 40, 45
    n = n0 + n_app
    w = WL.scaled(w0, n_tokens=n0)
    dev = torch.device("cuda")
    L, Bn, H, Hq = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads
    cache = B.Cache(L, Bn, H, Hq, w0.n_tokens + 64, device=dev, meta_format=meta_format, schedule=CAP)
    mod_cpu = WL.modality_layout(w)
    mod = mod_cpu.unsqueeze(0).repeat(Bn, 1).contiguous().to(dev)
    signs = torch.stack([WL.gen_signs(w, l) for l in range(L)])
    R = torch.stack([WL.gen_rotations(w, l) for l in range(L)])
    q = torch.stack([WL.gen_queries(w, l) for l in range(L)])
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
    new_k, new_v = [], []
    for s in range(n_app):
        kn, vn, mn = WL.gen_new_token(w, 0, s, device=dev)
        new_k.append(kn.cpu()); new_v.append(vn.cpu())
        B.append(cache, 0, L, kn.unsqueeze(0).expand(L, -1, -1, -1).contiguous(), vn.unsqueeze(0).expand(L, -1, -1, -1).contiguous(),
                 mn, d_signs, d_R)
    ws = torch.empty(B.decode_workspace_bytes(cache, L, 0), dtype=torch.uint8, device=dev)
    out = torch.full((L, Bn, Hq, D), float("nan"), dtype=torch.float32, device=dev)
    B.decode_attention(cache, 0, L, q.to(dev), d_signs, d_R, ws, out)
    torch.cuda.synchronize()
    assert cache.device_status() == 0 and (cache.seq_len == n).all()
    o = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(o).all()
    tail_k, tail_v = torch.stack(new_k, dim=2), torch.stack(new_v, dim=2)         # [B, H, n_app, 128]
    full = {key: (torch.cat([kc, tail_k[key[1]]], dim=1), torch.cat([vc, tail_v[key[1]]], dim=1)) for key, (kc, vc) in kept.items()}
    mod_row = np.concatenate([mod_cpu.numpy(), np.zeros(n_app, np.uint8)])
    _check_sampled(cache, w, samples, full, q, signs, R, mod_row, n, o, meta_format)
