"""Randomised parity sweep: shapes, lengths, GQA group sizes, metadata format, streaming schedule, shared or
per-head rotations and both value quantisers drawn from a seeded generator; every case compares the packed
cache (where the schedule has packed it) bit for bit and the decode output within the attention tolerance
against the oracle's definition."""
import numpy as np
import pytest
import torch

from oracle import okq_oracle as O
from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL
from tests import harness as Hn

pytestmark = pytest.mark.gpu
D, W = 128, 32


def _run_case(seed):
    rng = np.random.default_rng(1000 + seed)
    batch, hkv, group = int(rng.integers(1, 4)), int(rng.integers(1, 4)), int(rng.integers(1, 9))
    n = int(rng.choice([int(rng.integers(1, 40)), int(rng.integers(40, 300)), int(rng.integers(300, 900))]))
    meta_format, schedule = int(rng.integers(0, 2)), int(rng.integers(0, 2))
    per_head, bulk = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=batch, n_kv_heads=hkv, n_q_heads=hkv * group, n_tokens=n)
    g = torch.Generator().manual_seed(seed)
    k, v = WL.gen_kv(w, seed % 5, n_tokens=n)
    q = WL.gen_queries(w, seed % 5)
    signs = WL.gen_signs(w, seed % 5)
    n_R = hkv if per_head else 1
    R = torch.stack([WL.gen_rotations(w, (seed + 7 * r) % 11) for r in range(n_R)])          # [n_R, 3, 128, 128]
    mod = torch.randint(0, 3, (batch, n), generator=g, dtype=torch.uint8) if rng.integers(0, 2) else \
        WL.modality_layout(w, n)[None].repeat(batch, 1).contiguous()
    cap = ((n + 31) // 32 + 1) * 32
    cache = B.Cache(1, batch, hkv, hkv * group, cap, meta_format=meta_format, schedule=schedule)
    B.quantize_keys(cache, 0, k.cuda(), signs.cuda())
    B.quantize_values(cache, 0, v.cuda(), mod.cuda(), R.cuda(), bulk=bulk)
    ws = torch.empty(max(16, B.decode_workspace_bytes(cache, 1, 0)), dtype=torch.uint8, device="cuda")
    out = torch.full((1, batch, hkv * group, D), float("nan"), dtype=torch.float32, device="cuda")
    B.decode_attention(cache, 0, 1, q.cuda()[None], signs.cuda()[None], R.cuda()[None], ws, out, n_R=n_R)
    torch.cuda.synchronize()
    assert cache.device_status() == 0
    e = {a: x.cpu() for a, x in B.cache_export(cache, 0).items()}
    kp, vp = O.packed_counts(n, schedule)
    got = out[0].cpu().numpy().astype(np.float64)
    ref = np.zeros_like(got)
    for b in range(batch):
        for h in range(hkv):
            Rh = R[h if per_head else 0].numpy()
            kb, vb = Hn.u16(k[b, h]), Hn.u16(v[b, h])
            kq, vq, _ = O.quantize_batch(kb[None], vb[None], mod[b].numpy(), signs.numpy(), Rh, meta_format=meta_format)
            kq1 = {a: x[0] for a, x in kq.items()}; vq1 = {a: x[0] for a, x in vq.items()}
            assert (e["k_codes"][b, h, :kp].numpy() == kq1["codes"][:kp]).all(), "key codes"
            assert (Hn.u16(e["k_norm"][b, h, :kp]) == kq1["norm"][:kp]).all(), "key norms"
            assert (Hn.u16(e["k_meta"][b, h, :kp // W]) == kq1["meta"][:kp // W]).all(), "key (m, s)"
            assert (Hn.u16(e["v_norm"][b, h, :vp]) == vq1["norm"][:vp]).all(), "value norms"
            vc = e["v_codes"][b, h, :vp].numpy()
            if bulk:   # a coordinate on a codebook threshold may take the neighbouring level: use the stored codes
                assert (vc != vq1["codes"][:vp]).sum() <= 2
                vq1 = dict(vq1); vq1["codes"] = np.concatenate([vc, vq1["codes"][vp:]])
            else:
                assert (vc == vq1["codes"][:vp]).all(), "value codes"
            ref[b, h * group:(h + 1) * group] = O.attention_scheduled(
                Hn.u16(q[b, h * group:(h + 1) * group]), kq1, vq1, mod[b].numpy(), kb, vb, signs.numpy(), Rh, kp, vp)
    Hn.assert_attention_close(got, ref)
    return dict(batch=batch, hkv=hkv, group=group, n=n, meta=meta_format, schedule=schedule, per_head=per_head, bulk=bulk)


@pytest.mark.parametrize("seed", range(24))
def test_random_case(seed):
    print(_run_case(seed))
