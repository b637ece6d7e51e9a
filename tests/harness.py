"""Shared helpers of the GPU parity tests: build a cache with the CUDA library, build the
same cache with the CPU oracle, compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import okq_oracle as O
from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL

D, W = 128, 32
REL_L2_TOL = 1e-3      # attention output: relative L2 over the tensor and per (sequence, head) vector
MAX_ABS_TOL = 5e-3


def u16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


class Case:
    """One workload instantiated on the GPU (all layers) with per-layer inputs kept on the host."""

    def __init__(self, w: WL.Workload, n_tokens=None, capacity=None, device="cuda", gen_device="cpu",
                 meta_format=0, bulk_values=False, modality=None):
        self.w = w
        self.meta_format = meta_format
        self.n = w.n_tokens if n_tokens is None else n_tokens
        cap = capacity if capacity is not None else ((self.n + W - 1) // W + 2) * W
        self.cache = B.Cache(w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, cap, device=device,
                             meta_format=meta_format)
        self.mod = WL.modality_layout(w, self.n) if modality is None else modality   # [n]
        self.mod_b = self.mod.unsqueeze(0).repeat(w.batch, 1).contiguous()  # [B, n], as the caller passes it
        self.signs = torch.stack([WL.gen_signs(w, l) for l in range(w.n_layers)])      # [L,128]
        self.R = torch.stack([WL.gen_rotations(w, l) for l in range(w.n_layers)])      # [L,3,128,128]
        self.q = torch.stack([WL.gen_queries(w, l) for l in range(w.n_layers)])        # [L,B,Hq,128]
        self.k, self.v = [], []
        self.d_signs = self.signs.to(device)
        self.d_R = self.R.unsqueeze(1).contiguous().to(device)     # [L,1,3,128,128]
        self.d_q = self.q.to(device)
        self.d_mod = self.mod_b.to(device)
        for l in range(w.n_layers):
            k, v = WL.gen_kv(w, l, device=gen_device, n_tokens=self.n)
            self.k.append(k.cpu()); self.v.append(v.cpu())
            B.quantize_keys(self.cache, l, k.to(device), self.d_signs[l])
            B.quantize_values(self.cache, l, v.to(device), self.d_mod, self.d_R[l], bulk=bulk_values)
        torch.cuda.synchronize()

    # ---- oracle side
    @property
    def mod_o(self):
        """Modality ids as the oracle takes them ({0, 1, 2}: ids > 2 count as text), from the current mod_b."""
        return torch.where(self.mod_b > 2, torch.zeros_like(self.mod_b), self.mod_b).numpy()

    def oracle_quantize(self, layer):
        w = self.w
        U = w.batch * w.n_kv_heads
        kb = u16(self.k[layer]).reshape(U, self.n, D)
        vb = u16(self.v[layer]).reshape(U, self.n, D)
        unit_seq = np.repeat(np.arange(w.batch), w.n_kv_heads)
        kq, vq, _ = O.quantize_batch(kb, vb, self.mod_o, self.signs[layer].numpy(), self.R[layer].numpy(),
                                     unit_seq=unit_seq, meta_format=self.meta_format)
        return kq, vq, kb, vb

    def oracle_attention(self, layer, path=1, extra_k=None, extra_v=None, v_codes=None):
        """Oracle output [B, Hq, 128] for the bulk-built cache of `layer`.  `v_codes` (canonical value codes
        [B, Hkv, capacity, 32] as exported) replaces the oracle's own value codes: the tensor-core value
        quantiser may move a coordinate that sits on a codebook threshold to the neighbouring level."""
        w = self.w
        kq, vq, kb, vb = self.oracle_quantize(layer)
        if v_codes is not None:
            npk_ = (self.n // W) * W
            vq = dict(vq)
            vq["codes"] = np.ascontiguousarray(
                v_codes.cpu().numpy().reshape(w.batch * w.n_kv_heads, -1, 32)[:, :npk_])
        npk = (self.n // W) * W
        U = w.batch * w.n_kv_heads
        G = w.group
        q = u16(self.q[layer]).reshape(w.batch, w.n_kv_heads, G, D).reshape(U, G, D)
        unit_seq = np.repeat(np.arange(w.batch), w.n_kv_heads)
        out, th = O.attention(path, q, kq, vq, self.mod_o, kb[:, npk:], vb[:, npk:], self.signs[layer].numpy(),
                              self.R[layer].numpy(), unit_seq=unit_seq)
        return out.reshape(w.batch, w.n_q_heads, D), th

    # ---- GPU side
    def gpu_export(self, layer):
        e = B.cache_export(self.cache, layer)
        torch.cuda.synchronize()
        return e

    def gpu_decode(self, layer, layer_count=1, num_splits=0, simt=False):
        c = self.cache
        ws = torch.empty(max(16, B.decode_workspace_bytes(c, layer_count, num_splits)), dtype=torch.uint8, device=c.device)
        out = torch.full((layer_count, c.batch, c.n_q_heads, D), float("nan"), dtype=torch.float32, device=c.device)
        B.decode_attention(c, layer, layer_count, self.d_q[layer:layer + layer_count].contiguous(),
                           self.d_signs[layer:layer + layer_count].contiguous(),
                           self.d_R[layer:layer + layer_count].contiguous(), ws, out, num_splits=num_splits, simt=simt)
        torch.cuda.synchronize()
        return out.cpu().numpy().astype(np.float64)


def compare_cache(case: Case, layer: int, exp: dict, kq: dict, vq: dict):
    """Bit-exact comparison of the exported canonical arrays with the oracle's."""
    w = case.w
    npk = (case.n // W) * W
    U = w.batch * w.n_kv_heads
    cap = case.cache.capacity
    g = {k: v.cpu() for k, v in exp.items()}
    kc = g["k_codes"].numpy().reshape(U, cap, 32)[:, :npk]
    vc = g["v_codes"].numpy().reshape(U, cap, 32)[:, :npk]
    kn = u16(g["k_norm"]).reshape(U, cap)[:, :npk]
    vn = u16(g["v_norm"]).reshape(U, cap)[:, :npk]
    km = u16(g["k_meta"]).reshape(U, cap // W, D, 2)[:, :npk // W]
    assert (kn == kq["norm"]).all(), "key norms differ"
    assert (km == kq["meta"]).all(), f"key (m, s) differ at {np.argwhere(km != kq['meta'])[:4]}"
    assert (kc == kq["codes"]).all(), f"key codes differ: {(kc != kq['codes']).sum()} bytes"
    assert (vn == vq["norm"]).all(), "value norms differ"
    assert (vc == vq["codes"]).all(), f"value codes differ: {(vc != vq['codes']).sum()} bytes"
    if "mx" in kq:   # stored MXFP4 metadata bytes
        mx = g["k_mx"].numpy().reshape(U, cap // W, 136)[:, :npk // W]
        assert (mx == kq["mx"]).all(), f"stored MXFP4 metadata differs at {np.argwhere(mx != kq['mx'])[:4]}"


def attention_errors(got: np.ndarray, ref: np.ndarray):
    """(relative L2 over the tensor, worst relative L2 over (sequence, head) vectors, max abs)."""
    diff = got - ref
    rel = np.linalg.norm(diff) / np.linalg.norm(ref)
    per = np.linalg.norm(diff, axis=-1) / np.linalg.norm(ref, axis=-1)
    return rel, per.max(), np.abs(diff).max()


def assert_attention_close(got, ref):
    rel, worst, mx = attention_errors(got, ref)
    assert np.isfinite(got).all()
    assert rel < REL_L2_TOL and worst < REL_L2_TOL and mx < MAX_ABS_TOL, (rel, worst, mx)
    return rel, worst, mx
