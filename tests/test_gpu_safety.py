"""Stand-ins for a memory checker (none is available on the test machines): guard words around every
buffer the kernels write, and run-to-run bitwise determinism."""
import numpy as np
import pytest
import torch

from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL

pytestmark = pytest.mark.gpu
D, W = 128, 32
GUARD = 4096          # bytes of sentinel on each side
SENT = 0xA5


def _guarded(nbytes, dev):
    """uint8 buffer of nbytes with GUARD sentinel bytes before and after; returns (whole, view)."""
    pad = (-nbytes) % 16
    whole = torch.full((GUARD + nbytes + pad + GUARD,), SENT, dtype=torch.uint8, device=dev)
    return whole, whole[GUARD:GUARD + nbytes]


def _intact(whole, nbytes):
    pad = (-nbytes) % 16
    head, tail = whole[:GUARD], whole[GUARD + nbytes + pad:]
    return bool((head == SENT).all()) and bool((tail == SENT).all())


def test_guard_words_and_determinism():
    w = WL.scaled(WL.WORKLOADS["layer7b"], n_layers=2, batch=3, n_tokens=700 + 30)
    dev = torch.device("cuda")
    cap = 768
    L, Bn, H, Hq, N = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.n_tokens
    sizes = B.cache_sizes(L, Bn, H, Hq, cap)
    cache = B.Cache(L, Bn, H, Hq, cap, device=dev)
    # re-home every cache buffer inside guarded allocations
    names = ["records", "modality", "k_tail", "v_tail", "seq_len", "status"]
    guards = {}
    for name, nb in zip(names, sizes):
        whole, view = _guarded(nb, dev)
        view.zero_()
        guards[name] = (whole, nb)
        setattr(cache.c, name, view.data_ptr())
    rec_view = guards["records"][0][GUARD:GUARD + sizes[0]]
    seq_view = guards["seq_len"][0][GUARD:GUARD + sizes[4]].view(torch.int32)
    st_view = guards["status"][0][GUARD:GUARD + 4].view(torch.int32)

    mod = WL.modality_layout(w).unsqueeze(0).repeat(Bn, 1).contiguous().to(dev)
    signs = torch.stack([WL.gen_signs(w, l) for l in range(L)]).to(dev)
    R = torch.stack([WL.gen_rotations(w, l) for l in range(L)]).unsqueeze(1).contiguous().to(dev)
    q = torch.stack([WL.gen_queries(w, l) for l in range(L)]).to(dev)
    for l in range(L):
        k, v = WL.gen_kv(w, l, device=dev)
        B.quantize_keys(cache, l, k, signs[l])
        B.quantize_values(cache, l, v, mod, R[l], bulk=(l == 1))     # one layer through each value path
    for s in range(3):                                               # crosses a window boundary: one flush
        kn, vn, mn = WL.gen_new_token(w, 0, s, device=dev)
        kn = kn.unsqueeze(0).expand(L, -1, -1, -1).contiguous(); vn = vn.unsqueeze(0).expand(L, -1, -1, -1).contiguous()
        B.append(cache, 0, L, kn, vn, mn, signs, R)
    torch.cuda.synchronize()
    assert int(st_view[0]) == 0 and (seq_view == N + 3).all()

    ws_bytes = B.decode_workspace_bytes(cache, L, 0)
    ws_whole, ws = _guarded(ws_bytes, dev)
    out_bytes = L * Bn * Hq * D * 4
    outs = []
    for rep in range(3):
        o_whole, o = _guarded(out_bytes, dev)
        out = o.view(torch.float32).view(L, Bn, Hq, D)
        B.decode_attention(cache, 0, L, q, signs, R, ws, out)
        torch.cuda.synchronize()
        assert _intact(o_whole, out_bytes), "decode wrote outside its output"
        outs.append(out.clone())
    assert _intact(ws_whole, ws_bytes), "decode wrote outside its workspace"
    for name, (whole, nb) in guards.items():
        assert _intact(whole, nb), f"a kernel wrote outside the cache buffer `{name}`"
    # bitwise determinism of the whole path (no atomics on data, fixed merge order)
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[1], outs[2])
    assert torch.isfinite(outs[0]).all()
    # the CUDA-core kernel too
    s_whole, so = _guarded(out_bytes, dev)
    B.decode_attention(cache, 0, L, q, signs, R, ws, so.view(torch.float32).view(L, Bn, Hq, D), simt=True)
    torch.cuda.synchronize()
    assert _intact(s_whole, out_bytes) and _intact(ws_whole, ws_bytes)
    # export stays inside its arrays
    e = B.cache_export(cache, 0)
    torch.cuda.synchronize()
    assert e["k_codes"].shape == (Bn, H, cap, 32)
    del rec_view


def test_bounded_wait_runs_out_and_reports_timeout():
    """The tensor-core value quantiser with its first tile withheld and every wait limited to about ten milliseconds:
    each role's wait for that tile runs out, the kernel returns by itself and the device status word says
    ERR_TIMEOUT.  Nothing faults: the context stays usable, and the same call without the handicap then gives the
    codes of the exact quantiser."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=2)
    n = 1024 + 40
    dev = torch.device("cuda")
    k, v = WL.gen_kv(w, 0, n_tokens=n)
    mod = WL.modality_layout(w, n).unsqueeze(0).repeat(w.batch, 1).contiguous().to(dev)
    R = WL.gen_rotations(w, 0)[None].contiguous().to(dev)
    vd = v.to(dev)
    cache = B.Cache(1, w.batch, w.n_kv_heads, w.n_q_heads, 1088, device=dev)
    B.debug_bulk_timeout(cache, 0, vd, mod, R, limit_clocks=20_000_000)
    torch.cuda.synchronize()                      # returns: the kernel ended by itself
    assert cache.device_status() == B.ERR_TIMEOUT
    assert b"timed out" in B.lib().okq_status_string(B.ERR_TIMEOUT)
    cache.status.zero_()
    B.quantize_values(cache, 0, vd, mod, R, bulk=True)
    torch.cuda.synchronize()
    assert cache.device_status() == 0
    exact = B.Cache(1, w.batch, w.n_kv_heads, w.n_q_heads, 1088, device=dev)
    B.quantize_values(exact, 0, vd, mod, R)
    torch.cuda.synchronize()
    ea, eb = B.cache_export(cache, 0), B.cache_export(exact, 0)
    npk = (n // W) * W
    assert torch.equal(ea["v_codes"][:, :, :npk], eb["v_codes"][:, :, :npk]) and torch.equal(ea["v_norm"][:, :, :npk], eb["v_norm"][:, :, :npk])
