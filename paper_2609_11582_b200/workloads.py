"""Seeded synthetic workloads shaped like Qwen-Omni audio-visual decode caches.

This module only draws random inputs (keys, values, queries, modality ids,
Hadamard signs, orthogonal matrices).  It holds none of the quantiser's or the
attention kernel's arithmetic, so both the CUDA path and the CPU oracle can be
fed from it without sharing code.

The interleaved layout follows the paper's sequence structure
X = [V_1, A_1, ..., V_T, A_T, L] (Preliminaries, before Eq. 1): video tokens then
audio tokens per 2-second chunk, surrounded by text.  350 tokens per chunk is
10 500 tokens per minute, the scale the Introduction quotes (>10 000 per minute).

Statistics (chosen so that 32-token windows of rotated keys are much narrower
than the global distribution, the effect Table 1 reports):
  keys    k[i,c] = a[c] * (mu[i,c] + eps[i,c]),  mu a Gaussian random walk over
          time with step sigma 0.05 starting from N(0,1), eps ~ N(0,1),
          a[c] = 10 on 4 seeded outlier channels and 1 elsewhere.
  values  v = Q_m g + 0.1 eps with Q_m a seeded 128x16 orthonormal frame per
          modality, g ~ N(0, I_16), eps ~ N(0, I_128).
  queries N(0,1).   R_m: Haar orthogonal (QR of a Gaussian matrix with sign
  fix).  D: seeded +-1 signs.
All tensors are drawn in float32 (rotations in float64) and cast to fp16.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

TEXT, AUDIO, VIDEO = 0, 1, 2
HEAD_DIM = 128
WINDOW = 32


@dataclass(frozen=True)
class Workload:
    name: str
    index: int            # position in the benchmark's config list (used in seeds)
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    n_tokens: int
    prefix_text: int
    video_chunk: int
    audio_chunk: int
    suffix_text: int
    n_chunks: int = 0     # 0: repeat chunks until the suffix; >0: exactly this many

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def token_heads(self) -> int:
        return self.n_layers * self.batch * self.n_kv_heads * self.n_tokens


WORKLOADS = {
    # tiny single-head decode: [text 64 | (video 180, audio 50) x 8 | text 144] = 2048
    "tiny": Workload("tiny", 0, 1, 1, 7, 1, 2048, 64, 180, 50, 144, 8),
    # 7B-shaped single layer, 8192 tokens
    "layer7b": Workload("layer7b", 1, 1, 1, 28, 4, 8192, 128, 300, 50, 64),
    # 7B-shaped full decode step: 28 layers, batch 8, 16k context
    "step7b": Workload("step7b", 2, 28, 8, 28, 4, 16384, 128, 300, 50, 64),
    # 30B-A3B-shaped decode attention: 48 layers, batch 16, 32k context
    "step30b": Workload("step30b", 3, 48, 16, 32, 4, 32768, 256, 400, 100, 0),
    # prefill quantisation of 32k tokens, 7B shape, batch 1
    "prefill7b": Workload("prefill7b", 4, 28, 1, 28, 4, 32768, 128, 300, 50, 64),
    # long-context decode, batch 1 at 131072
    "long7b": Workload("long7b", 4, 28, 1, 28, 4, 131072, 128, 300, 50, 64),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (used for reduced test sizes)."""
    d = dict(w.__dict__)
    d.update(kw)
    return Workload(**d)


def modality_layout(w: Workload, n_tokens: int | None = None) -> torch.Tensor:
    """uint8 [n_tokens]: 0 text, 1 audio, 2 video, in the interleaved chunk order."""
    n = w.n_tokens if n_tokens is None else n_tokens
    mod = torch.empty(n, dtype=torch.uint8)
    pos = min(w.prefix_text, n)
    mod[:pos] = TEXT
    body_end = n - w.suffix_text if w.n_chunks == 0 else n
    body_end = max(body_end, pos)
    chunks = 0
    while pos < body_end and (w.n_chunks == 0 or chunks < w.n_chunks):
        e = min(pos + w.video_chunk, body_end)
        mod[pos:e] = VIDEO
        pos = e
        e = min(pos + w.audio_chunk, body_end)
        mod[pos:e] = AUDIO
        pos = e
        chunks += 1
    mod[pos:] = TEXT
    return mod


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _seed(w: Workload, layer: int, stream: int) -> int:
    return 20260911 + 1000 * w.index + layer + 7919 * stream


def gen_signs(w: Workload, layer: int) -> torch.Tensor:
    """float32 [128] of +-1: the diagonal D of the randomised Hadamard transform."""
    g = _gen("cpu", _seed(w, layer, 1))
    return (torch.randint(0, 2, (HEAD_DIM,), generator=g).to(torch.float32) * 2 - 1)


def gen_rotations(w: Workload, layer: int) -> torch.Tensor:
    """float32 [3,128,128] Haar-distributed orthogonal matrices, index = modality id."""
    g = _gen("cpu", _seed(w, layer, 2))
    out = []
    for _ in range(3):
        a = torch.randn(HEAD_DIM, HEAD_DIM, generator=g, dtype=torch.float64)
        q, r = torch.linalg.qr(a)
        q = q * torch.sign(torch.diagonal(r)).unsqueeze(0)
        out.append(q)
    return torch.stack(out).to(torch.float32).contiguous()


def gen_queries(w: Workload, layer: int, device="cpu") -> torch.Tensor:
    """fp16 [batch, n_q_heads, 128] ~ N(0,1)."""
    g = _gen(device, _seed(w, layer, 3))
    q = torch.randn(w.batch, w.n_q_heads, HEAD_DIM, generator=g, device=device, dtype=torch.float32)
    return q.to(torch.float16)


def gen_kv(w: Workload, layer: int, device="cpu", n_tokens: int | None = None,
           seqs: slice | None = None):
    """Keys and values of one layer: two fp16 tensors [batch, n_kv_heads, n_tokens, 128].

    `seqs` restricts the batch to a slice (each sequence has its own seed, so a
    slice reproduces exactly the rows of the full batch).
    """
    n = w.n_tokens if n_tokens is None else n_tokens
    mod = modality_layout(w, n).to(device)
    rng = range(w.batch)[seqs] if seqs is not None else range(w.batch)
    ks, vs = [], []
    for b in rng:
        g = _gen(device, _seed(w, layer, 10 + b))
        H = w.n_kv_heads
        mu0 = torch.randn(H, 1, HEAD_DIM, generator=g, device=device)
        steps = torch.randn(H, n, HEAD_DIM, generator=g, device=device) * 0.05
        steps[:, :1, :] = 0
        mu = mu0 + torch.cumsum(steps, dim=1)
        del steps
        k = mu + torch.randn(H, n, HEAD_DIM, generator=g, device=device)
        del mu
        amp = torch.ones(H, HEAD_DIM, device=device)
        for h in range(H):
            idx = torch.randperm(HEAD_DIM, generator=g, device=device)[:4]
            amp[h, idx] = 10.0
        k = (k * amp.unsqueeze(1)).to(torch.float16)
        # values: per modality rank-16 subspace + isotropic noise
        frames = torch.randn(H, 3, HEAD_DIM, 16, generator=g, device=device, dtype=torch.float32)
        frames, _ = torch.linalg.qr(frames)                      # orthonormal columns
        coef = torch.randn(H, n, 16, generator=g, device=device)
        v = torch.empty(H, n, HEAD_DIM, device=device)
        for m in range(3):
            sel = (mod == m).nonzero().squeeze(1)
            if sel.numel():
                v[:, sel] = torch.matmul(coef[:, sel], frames[:, m].transpose(1, 2))
        del coef
        v = v + 0.1 * torch.randn(H, n, HEAD_DIM, generator=g, device=device)
        ks.append(k)
        vs.append(v.to(torch.float16))
    return torch.stack(ks).contiguous(), torch.stack(vs).contiguous()


def gen_new_token(w: Workload, layer: int, step: int, device="cpu"):
    """One new text token per sequence: fp16 k, v [batch, n_kv_heads, 128], uint8 modality [batch]."""
    g = _gen(device, _seed(w, layer, 5000 + step))
    k = torch.randn(w.batch, w.n_kv_heads, HEAD_DIM, generator=g, device=device)
    v = torch.randn(w.batch, w.n_kv_heads, HEAD_DIM, generator=g, device=device) * 0.3
    mod = torch.zeros(w.batch, dtype=torch.uint8, device=device)
    return k.to(torch.float16), v.to(torch.float16), mod
