#!/usr/bin/env python
"""Benchmark of the okq hot path: one decode step = okq_append of one new text token per
sequence to every layer + okq_decode_attention over every layer's packed cache.

Default workload: the 7B-shaped full decode step (28 layers, 28/4 heads, batch 8, 16384
tokens of context per sequence), synthetic seeded inputs.  Prints ONE JSON line.

  value        packed-KV bytes of the step / device time of the step (GB/s), whole job
  e2e          the same with this step's queries / new tokens copied from pinned host memory
               and the attention output copied back, inside the timed region
  roofline     the split-K decode kernel alone (CUDA events recorded around it on its stream)
  cpu_baseline the CPU oracle timed on a bounded sample of the same workload

`--impl reference` times the CPU oracle (the only reference this method has) instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_11582_b200 import workloads as WL  # noqa: E402

METRIC = "2-bit KV decode-attention effective HBM GB/s (packed-KV bytes per decode step / step time)"
W_TOKENS = 32                      # tokens per window: one step in 32 packs a window ("flush")
BYTES_PER_TOKEN_HEAD = 84          # 32 B key codes + 2 B key norm + 16 B (m, s) + 32 B value codes + 2 B value norm
# dram__bytes_read.sum + dram__bytes_write.sum of one split-K decode launch, measured with ncu on a
# 4-layer slice of the workload (176 MB of records, larger than L2) and divided by its token-heads;
# traffic grows in proportion to the token-heads.  To be re-measured whenever the split-K kernel changes.
NCU_DRAM_BYTES_PER_TOKEN_HEAD = 86.36
NCU_DRAM_BYTES_PER_TOKEN_HEAD_MX = 74.82   # same capture with --meta mxfp4


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Reads SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def oracle_prepare(w, n_layers_s, n_seq_s):
    """Inputs of the CPU oracle for n_layers_s x n_seq_s sequences of the workload (the oracle
    quantises the sampled fp16 inputs itself).  Returns (attention args, unit_rot, token-heads)."""
    from oracle import okq_oracle as O
    mod = WL.modality_layout(w).numpy()
    kqs, vqs, qs, signs, Rs, kt, vt = [], [], [], [], [], [], []
    U_per = n_seq_s * w.n_kv_heads
    for l in range(n_layers_s):
        k, v = WL.gen_kv(w, l, device="cpu", seqs=slice(0, n_seq_s))
        kb = k.view(torch.int16).numpy().view(np.uint16).reshape(U_per, w.n_tokens, 128)
        vb = v.view(torch.int16).numpy().view(np.uint16).reshape(U_per, w.n_tokens, 128)
        sg = WL.gen_signs(w, l).numpy(); R = WL.gen_rotations(w, l).numpy()
        kq, vq, _ = O.quantize_batch(kb, vb, mod, sg, R)
        kqs.append(kq); vqs.append(vq); signs.append(sg); Rs.append(R)
        q = WL.gen_queries(w, l)[:n_seq_s].view(torch.int16).numpy().view(np.uint16)
        qs.append(q.reshape(n_seq_s, w.n_kv_heads, w.group, 128).reshape(U_per, w.group, 128))
        npk = (w.n_tokens // 32) * 32
        kt.append(kb[:, npk:]); vt.append(vb[:, npk:])
    cat = lambda ds, key: np.concatenate([d[key] for d in ds])
    kq = {k: cat(kqs, k) for k in ("codes", "norm", "meta")}
    vq = {k: cat(vqs, k) for k in ("codes", "norm")}
    unit_rot = np.repeat(np.arange(n_layers_s), U_per)
    args = (np.concatenate(qs), kq, vq, mod, np.concatenate(kt), np.concatenate(vt), np.stack(signs), np.stack(Rs))
    return args, unit_rot, n_layers_s * U_per * w.n_tokens


def oracle_pass(args, unit_rot):
    """One timed pass of the oracle's rotated-space attention; returns (seconds, threads)."""
    from oracle import okq_oracle as O
    t0 = time.perf_counter()
    _, th = O.attention(1, *args, unit_rot=unit_rot)
    return time.perf_counter() - t0, th


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    # a bounded sample per "step": one oracle attention pass over 1 layer x 4 sequences
    n_seq_s = min(4, w.batch)
    oargs, unit_rot, th_units = oracle_prepare(w, 1, n_seq_s)
    per_step, threads = [], 1
    for _ in range(args.warmup + args.steps):
        t, threads = oracle_pass(oargs, unit_rot)
        per_step.append(t)
    ts = per_step[args.warmup:]
    t = sum(ts) / len(ts)
    gbs = th_units * BYTES_PER_TOKEN_HEAD / t / 1e9
    sample = (f"1 layer x {n_seq_s} sequences x {w.n_kv_heads} KV heads x {w.n_tokens} tokens per step "
              "(oracle rotated-space attention; GB/s = packed bytes of the sample / time)")
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "n_layers": w.n_layers, "batch": w.batch, "n_q_heads": w.n_q_heads,
                       "n_kv_heads": w.n_kv_heads, "context": w.n_tokens, "sample": sample},
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_prefill(args, w, B, dev, rank, emit=True):
    """Secondary measurement: bulk okq_quantize_keys + okq_quantize_values_bulk over a fresh fp16 K/V cache of
    every layer (the prefill half of the long-context configuration).  One JSON line (or, emit=False, the dict)."""
    L, Bn, H, Hq, N = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.n_tokens
    cache = B.Cache(L, Bn, H, Hq, N, device=dev)
    mod = WL.modality_layout(w).unsqueeze(0).repeat(Bn, 1).contiguous().to(dev)
    signs = torch.stack([WL.gen_signs(w, l) for l in range(L)]).to(dev)
    R = torch.stack([WL.gen_rotations(w, l) for l in range(L)]).unsqueeze(1).contiguous().to(dev)
    kv = [WL.gen_kv(w, l, device=dev) for l in range(L)]
    th = L * Bn * H * N
    in_bytes, out_bytes = th * 512, th * BYTES_PER_TOKEN_HEAD

    def timed(fn):
        for _ in range(args.warmup):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in ev:
            a.record(); fn(); b.record()
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev) / args.steps

    ms_k = timed(lambda: [B.quantize_keys(cache, l, kv[l][0], signs[l]) for l in range(L)])
    ms_v = timed(lambda: [B.quantize_values(cache, l, kv[l][1], mod, R[l], bulk=True) for l in range(L)])
    ms_vx = timed(lambda: [B.quantize_values(cache, l, kv[l][1], mod, R[l]) for l in range(min(L, 2))]) * L / min(L, 2)
    if cache.device_status() != 0:
        raise RuntimeError("device status word set during the benchmark")
    peak, peak_kind = measured_peaks()
    ms = ms_k + ms_v
    line = {"metric": "prefill quantisation: fp16 K/V bytes in + packed bytes out per second", "phase": "prefill",
            "value": (in_bytes + out_bytes) / (ms * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "dtype": "f32/f16-mma", "data": "synthetic",
            "config": {"workload": w.name, "n_layers": L, "batch": Bn, "n_kv_heads": H, "context": N},
            "keys_ms": ms_k, "values_bulk_ms": ms_v, "values_exact_ms_scaled": ms_vx,
            "keys_gbs": th * 306 / (ms_k * 1e-3) / 1e9, "values_bulk_gbs": th * 290 / (ms_v * 1e-3) / 1e9,
            "values_bulk_tflops": th * 2 * 2 * 128 * 128 / (ms_v * 1e-3) / 1e12,
            "roofline": {"bound": "hbm", "kernel": "key + value quantisers", "achieved": (in_bytes + out_bytes) / (ms * 1e-3) / 1e9,
                         "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                         "frac": (in_bytes + out_bytes) / (ms * 1e-3) / 1e9 / peak, "traffic": None}}
    del kv, cache
    if not emit:
        return line
    if rank == 0:
        print(json.dumps(line), flush=True)


def run_ladder(args, B, dev, rank, emit=True):
    """Secondary measurement: the bit-width ladder entry points (K2V2 / K3V3 / K4V4 over the canonical bit-stream
    cache; plain CUDA-core kernels, one thread block per (sequence, KV head) in decode) and the TurboQuant codec,
    on 256 sequences x 4 KV heads x 8192 tokens of the 7B layer shape (1024 thread blocks in decode).  GB/s of packed bytes read per decode."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=256, name="layer7b[batch=256]")
    Bn, H, Hq, N = w.batch, w.n_kv_heads, w.n_q_heads, w.n_tokens
    k, v = WL.gen_kv(w, 0, device=dev)
    q = WL.gen_queries(w, 0, device=dev)
    signs = WL.gen_signs(w, 0).to(dev)
    R = WL.gen_rotations(w, 0).unsqueeze(0).contiguous().to(dev)
    mod = WL.modality_layout(w).unsqueeze(0).repeat(Bn, 1).contiguous().to(dev)
    out = torch.empty((Bn, Hq, 128), dtype=torch.float32, device=dev)
    peak, peak_kind = measured_peaks()
    th = Bn * H * N

    def timed(fn):
        for _ in range(args.warmup):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in ev:
            a.record(); fn(); b.record()
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev) / args.steps

    res = {}
    for bits in (2, 3, 4):
        cache = B.LadderCache(Bn, H, Hq, N, bits, device=dev)
        ms_k = timed(lambda: B.ladder_quantize_keys(cache, k, signs))
        ms_v = timed(lambda: B.ladder_quantize_values(cache, v, mod, R))
        ms_d = timed(lambda: B.ladder_decode_attention(cache, N, q, signs, R, out))
        bytes_th = 2 * 16 * bits + 4 + 16            # codes, two fp16 norms, (m, s) of 128 channels per 32 tokens
        res[f"K{bits}V{bits}"] = {"bytes_per_token_head": bytes_th, "bits_per_element": bytes_th * 8 / 256,
                                  "quantize_keys_ms": ms_k, "quantize_values_ms": ms_v, "decode_ms": ms_d,
                                  "decode_gbs": th * bytes_th / (ms_d * 1e-3) / 1e9,
                                  "decode_frac": th * bytes_th / (ms_d * 1e-3) / 1e9 / peak}
        del cache
    x = k.reshape(-1, 128)
    ms_e = timed(lambda: B.turboquant_encode(x, signs, 2))
    codes, norms = B.turboquant_encode(x, signs, 2)
    ms_x = timed(lambda: B.turboquant_decode(codes, norms, signs, 2))
    res["turboquant_k2"] = {"encode_ms": ms_e, "decode_ms": ms_x, "encode_gbs": th * (256 + 34) / (ms_e * 1e-3) / 1e9}
    line = {"metric": "bit-width ladder decode attention: packed bytes per second", "phase": "ladder", "unit": "GB/s",
            "value": res["K4V4"]["decode_gbs"], "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": res["K4V4"]["decode_ms"], "higher_is_better": True, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "batch": Bn, "n_kv_heads": H, "context": N}, "peak": peak, "peak_kind": peak_kind,
            "ladder": res}
    if not emit:
        return line
    if rank == 0:
        print(json.dumps(line), flush=True)


def quick_decode(B, dev, w, mx=False, caption=False, steps=8, warmup=3):
    """Short secondary measurement of the decode step (append + decode over all layers, inputs resident) on another
    workload / metadata format / schedule: step time, GB/s of packed bytes, split-K kernel time and fraction."""
    L, Bn, H, Hq, N = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.n_tokens
    bytes_th = 72.25 if mx else BYTES_PER_TOKEN_HEAD
    cache = B.Cache(L, Bn, H, Hq, N + 64, device=dev, meta_format=B.META_MXFP4 if mx else B.META_FP16,
                    schedule=B.SCHEDULE_CAPTION if caption else B.SCHEDULE_WINDOW)
    mod = WL.modality_layout(w).unsqueeze(0).repeat(Bn, 1).contiguous().to(dev)
    signs = torch.stack([WL.gen_signs(w, l) for l in range(L)]).to(dev)
    R = torch.stack([WL.gen_rotations(w, l) for l in range(L)]).unsqueeze(1).contiguous().to(dev)
    for l in range(L):
        k, v = WL.gen_kv(w, l, device=dev)
        B.quantize_keys(cache, l, k, signs[l])
        B.quantize_values(cache, l, v, mod, R[l], bulk=True)
        del k, v
    torch.cuda.synchronize()
    seq0 = cache.seq_len.clone()
    q = torch.stack([WL.gen_queries(w, l) for l in range(L)]).to(dev)
    kn, vn, mn = WL.gen_new_token(w, 0, 0, device=dev)
    kn = kn.unsqueeze(0).expand(L, -1, -1, -1).contiguous(); vn = vn.unsqueeze(0).expand(L, -1, -1, -1).contiguous()
    out = torch.empty(L, Bn, Hq, 128, dtype=torch.float32, device=dev)
    ws = torch.empty(max(16, B.decode_workspace_bytes(cache, L, 0)), dtype=torch.uint8, device=dev)

    def step():
        B.append(cache, 0, L, kn, vn, mn, signs, R)
        B.decode_attention(cache, 0, L, q, signs, R, ws, out)
    for _ in range(warmup):
        step()
    cache.seq_len.copy_(seq0)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in kev:
        a.record(); b.record()
    torch.cuda.synchronize()
    for i in range(steps):
        B.profile_events(*kev[i])
        ev[i][0].record(); step(); ev[i][1].record()
    torch.cuda.synchronize()
    B.profile_events(None, None)
    if cache.device_status() != 0 or not torch.isfinite(out).all():
        raise RuntimeError("secondary decode measurement: bad device status or non-finite output")
    ms = sum(a.elapsed_time(b) for a, b in ev) / steps
    kms = sum(a.elapsed_time(b) for a, b in kev) / steps
    packed = L * Bn * H * N * bytes_th
    peak, _ = measured_peaks()
    return {"workload": w.name, "meta_format": "mxfp4" if mx else "fp16", "schedule": "caption" if caption else "window",
            "steps": steps, "us_per_step": ms * 1e3, "value": packed / (ms * 1e-3) / 1e9, "unit": "GB/s",
            "kernel_us": kms * 1e3, "kernel_gbs": packed / (kms * 1e-3) / 1e9, "kernel_frac": packed / (kms * 1e-3) / 1e9 / peak}


def run_calib(args, B, dev, rank):
    """Secondary measurement: the offline calibration of the value rotations of one (layer, KV head) on a
    synthetic calibration sequence of 8192 tokens (7 query heads): attention weights, weighted moments, three
    eigen-decompositions.  One JSON line."""
    n, G = 8192, 7
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=1, n_tokens=n)
    k, v = WL.gen_kv(w, 0, device=dev, n_tokens=n)
    k, v = k[0, 0].contiguous(), v[0, 0].contiguous()
    q = torch.randn(G, n, 128, generator=torch.Generator(device=dev).manual_seed(7), device=dev).to(torch.float16)
    mod = WL.modality_layout(w, n).to(dev)
    signs = WL.gen_signs(w, 0).to(dev)
    ws = B.calib_workspace(G, n, device=dev)

    def timed(fn):
        for _ in range(args.warmup):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in ev:
            a.record(); fn(); b.record()
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev) / args.steps

    wts = B.calib_attention_weights(q, k, ws)
    Cm = B.calib_moments(v, wts, mod, ws)
    ms_w = timed(lambda: B.calib_attention_weights(q, k, ws))
    ms_c = timed(lambda: B.calib_moments(v, wts, mod, ws))
    ms_r = timed(lambda: [B.calib_rotation(Cm[m].contiguous(), signs, ws) for m in range(3)])
    peak, peak_kind = measured_peaks()
    # causal scores, computed in both passes: 2 passes x G x n (n + 64) / 2 x 128 multiply-adds (64-key tiles)
    flops_w = 2.0 * 2 * G * n * (n + 64) / 2 * 128
    line = {"metric": "calibration of the value rotations: ms per (layer, KV head)", "phase": "calib",
            "value": ms_w + ms_c + ms_r, "unit": "ms", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "higher_is_better": False, "dtype": "f16-mma/f32/f64", "data": "synthetic",
            "config": {"workload": "calibration sequence", "tokens": n, "group": G},
            "attention_weights_ms": ms_w, "attention_weights_tflops": flops_w / (ms_w * 1e-3) / 1e12,
            "moments_ms": ms_c, "rotations_ms": ms_r}
    if rank == 0:
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="okq", choices=["okq", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(WL.WORKLOADS))
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--decode-kernel", default="default", choices=["default", "tcgen05", "mma"],
                    help="split-K kernel behind okq_decode_attention (default: the library's choice)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the short secondary measurements of the default run")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (profiling on a small case)")
    ap.add_argument("--meta", default="fp16", choices=["fp16", "mxfp4"],
                    help="(m, s) metadata format of the cache: fp16 = 84 B per token and KV head (the headline "
                         "configuration), mxfp4 = 72.25 B (secondary measurement; no cpu_baseline)")
    ap.add_argument("--schedule", default="window", choices=["window", "caption"],
                    help="streaming schedule of the cache: window = pack every 32 tokens (the headline configuration), "
                         "caption = the paper's captioning schedule (keys every 128 tokens, values behind a 128-token "
                         "fp16 window; secondary measurement, no cpu_baseline)")
    ap.add_argument("--phase", default="decode", choices=["decode", "prefill", "calib", "ladder"],
                    help="decode: the headline decode step; prefill: bulk quantisation of a fresh fp16 K/V cache "
                         "(secondary measurement, default workload prefill7b); calib: offline calibration of the "
                         "value rotations (secondary measurement); ladder: the K2V2 / K3V3 / K4V4 entry points and the "
                         "TurboQuant codec (secondary measurement)")
    args = ap.parse_args()
    if args.workload is None:
        args.workload = "prefill7b" if args.phase == "prefill" else "step7b"
    w = WL.WORKLOADS[args.workload]
    if args.layers > 0:
        w = WL.scaled(w, n_layers=args.layers, name=f"{w.name}[layers={args.layers}]")
    if args.impl == "reference":
        return run_reference(args, w)

    from paper_2609_11582_b200 import binding as B
    if args.decode_kernel != "default":
        B.decode_select(0 if args.decode_kernel == "tcgen05" else 1)
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    if args.phase == "prefill":
        return run_prefill(args, w, B, dev, rank)
    if args.phase == "calib":
        return run_calib(args, B, dev, rank)
    if args.phase == "ladder":
        return run_ladder(args, B, dev, rank)

    # ---- build the packed cache on the device (setup, untimed)
    L, Bn, H, Hq, N = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.n_tokens
    mx = args.meta == "mxfp4"
    bytes_th = 72.25 if mx else BYTES_PER_TOKEN_HEAD
    caption = args.schedule == "caption"
    cache = B.Cache(L, Bn, H, Hq, N + 64, device=dev, meta_format=B.META_MXFP4 if mx else B.META_FP16,
                    schedule=B.SCHEDULE_CAPTION if caption else B.SCHEDULE_WINDOW)
    mod = WL.modality_layout(w).unsqueeze(0).repeat(Bn, 1).contiguous().to(dev)
    signs = torch.stack([WL.gen_signs(w, l) for l in range(L)]).to(dev)
    R = torch.stack([WL.gen_rotations(w, l) for l in range(L)]).unsqueeze(1).contiguous().to(dev)
    for l in range(L):
        k, v = WL.gen_kv(w, l, device=dev)
        B.quantize_keys(cache, l, k, signs[l])
        B.quantize_values(cache, l, v, mod, R[l], bulk=True)   # prefill path: rotation on the tensor cores
        del k, v
    torch.cuda.synchronize()
    seq0 = cache.seq_len.clone()

    total = args.warmup + args.steps
    q_host = torch.stack([WL.gen_queries(w, l) for l in range(L)]).pin_memory()          # [L,B,Hq,128] fp16
    newtok = [WL.gen_new_token(w, 0, s) for s in range(total)]
    kn_host = torch.stack([t[0].unsqueeze(0).expand(L, -1, -1, -1) for t in newtok]).contiguous().pin_memory()
    vn_host = torch.stack([t[1].unsqueeze(0).expand(L, -1, -1, -1) for t in newtok]).contiguous().pin_memory()
    mn_host = torch.zeros(Bn, dtype=torch.uint8).pin_memory()
    out_host = torch.empty(L, Bn, Hq, 128, dtype=torch.float32).pin_memory()

    q_dev = q_host.to(dev); kn_dev = kn_host.to(dev); vn_dev = vn_host.to(dev); mn_dev = mn_host.to(dev)
    out = torch.empty(L, Bn, Hq, 128, dtype=torch.float32, device=dev)
    ws = torch.empty(max(16, B.decode_workspace_bytes(cache, L, args.splits)), dtype=torch.uint8, device=dev)
    packed_bytes = int(L * Bn * H * N * bytes_th)

    def step_resident(s):
        B.append(cache, 0, L, kn_dev[s], vn_dev[s], mn_dev, signs, R)
        B.decode_attention(cache, 0, L, q_dev, signs, R, ws, out, num_splits=args.splits)

    # End to end: every step's queries / new token cross PCIe from pinned host memory and its output goes
    # back, on a second stream with two sets of device buffers, so that the copies of neighbouring steps
    # overlap the kernels (the host API is asynchronous; this is how a caller would drive it).
    copy_stream = torch.cuda.Stream(device=dev)
    in_buf = [(torch.empty_like(q_dev), torch.empty_like(kn_dev[0]), torch.empty_like(vn_dev[0]), torch.empty_like(mn_dev))
              for _ in range(2)]
    out_buf = [torch.empty_like(out) for _ in range(2)]
    out_host2 = [torch.empty(L, Bn, Hq, 128, dtype=torch.float32).pin_memory() for _ in range(2)]

    def run_e2e(first, count):
        """`count` pipelined steps starting at input index `first`; returns when everything is enqueued."""
        main = torch.cuda.current_stream(dev)
        in_ready = [torch.cuda.Event(), torch.cuda.Event()]
        done = [torch.cuda.Event(), torch.cuda.Event()]

        def prefetch(i):
            qb, kb, vb, mb = in_buf[i & 1]
            with torch.cuda.stream(copy_stream):
                qb.copy_(q_host, non_blocking=True)
                kb.copy_(kn_host[first + i], non_blocking=True)
                vb.copy_(vn_host[first + i], non_blocking=True)
                mb.copy_(mn_host, non_blocking=True)
                in_ready[i & 1].record(copy_stream)

        copy_stream.wait_stream(main)
        prefetch(0)
        for i in range(count):
            qb, kb, vb, mb = in_buf[i & 1]
            main.wait_event(in_ready[i & 1])
            if i >= 2:
                main.wait_event(d2h_done[i & 1])      # out_buf[i & 1] has been read back
            B.append(cache, 0, L, kb, vb, mb, signs, R)
            B.decode_attention(cache, 0, L, qb, signs, R, ws, out_buf[i & 1], num_splits=args.splits)
            done[i & 1].record(main)
            if i + 1 < count:
                if i >= 1:
                    copy_stream.wait_event(done[(i - 1) & 1])   # in_buf[(i + 1) & 1] was last read by step i - 1
                prefetch(i + 1)
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(done[i & 1])
                out_host2[i & 1].copy_(out_buf[i & 1], non_blocking=True)
                d2h_done[i & 1].record(copy_stream)
        main.wait_stream(copy_stream)

    d2h_done = [torch.cuda.Event(), torch.cuda.Event()]

    def timed_e2e():
        cache.seq_len.copy_(seq0)
        run_e2e(0, args.warmup)
        prime()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record()
        run_e2e(args.warmup, args.steps)
        b.record()
        barrier()
        ms = a.elapsed_time(b)
        last = (args.steps - 1) & 1      # the read-back copy is the device result of the last step
        if not torch.equal(out_host2[last], out_buf[last].cpu()) or not torch.isfinite(out_host2[last]).all():
            raise RuntimeError("end-to-end run: host copy of the output differs from the device result")
        if world > 1:
            import torch.distributed as dist
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # The timed steps end on a 32-token boundary, so that whatever --steps is they contain a step that packs a
    # window (one per 32 steps): `pre` untimed appends put the raw tokens of the earlier steps of the cycle in place.
    pre = (-args.steps) % W_TOKENS

    def prime():
        cache.seq_len.copy_(seq0)
        for _ in range(pre):
            B.append(cache, 0, L, kn_dev[0], vn_dev[0], mn_dev, signs, R)

    def timed(step_fn, with_kernel_events):
        cache.seq_len.copy_(seq0)
        for s in range(args.warmup):
            step_fn(s)
        prime()                          # the timed steps always start from the same context length
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in kev:      # torch creates the CUDA event on first record; the library re-records it later
            a.record(); b.record()
        barrier()
        sampler = ClockSampler(local)
        sampler.start()
        for i in range(args.steps):
            if with_kernel_events:
                B.profile_events(*kev[i])
            ev[i][0].record()
            step_fn(args.warmup + i)
            ev[i][1].record()
        barrier()
        B.profile_events(None, None)
        clocks = sampler.stop()
        per_step = [a.elapsed_time(b) for a, b in ev]
        ms = sum(per_step)
        kms = sum(a.elapsed_time(b) for a, b in kev) / args.steps if with_kernel_events else None
        flush = [t for i, t in enumerate(per_step) if (pre + i + 1) % W_TOKENS == 0]
        tail = [t for i, t in enumerate(per_step) if (pre + i + 1) % W_TOKENS != 0]
        step_kinds.update(flush_steps=len(flush), us_per_flush_step=1e3 * sum(flush) / max(1, len(flush)),
                          tail_steps=len(tail), us_per_tail_step=1e3 * sum(tail) / max(1, len(tail)) if tail else None)
        if world > 1:
            import torch.distributed as dist
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms, kms, clocks

    step_kinds = {}
    ms_total, kernel_ms, clocks = timed(step_resident, True)
    if cache.device_status() != 0:
        raise RuntimeError("device status word set during the benchmark")
    ms_e2e = timed_e2e()
    ms_step = ms_total / args.steps
    value = world * packed_bytes / (ms_step * 1e-3) / 1e9
    e2e_value = world * packed_bytes / (ms_e2e / args.steps * 1e-3) / 1e9
    peak, peak_kind = measured_peaks()
    achieved = packed_bytes / (kernel_ms * 1e-3) / 1e9
    traffic = (NCU_DRAM_BYTES_PER_TOKEN_HEAD_MX if mx else NCU_DRAM_BYTES_PER_TOKEN_HEAD) * L * Bn * H * N

    # The same step as a model issues it: one okq_append + one okq_decode_attention per layer (2 L calls),
    # captured once in a CUDA graph and replayed, so that the launch gaps between the per-layer kernels count.
    def per_layer_graph_ms():
        def one_step():
            for l in range(L):
                B.append(cache, l, 1, kn_dev[0][l:l + 1], vn_dev[0][l:l + 1], mn_dev, signs[l:l + 1], R[l:l + 1])
                B.decode_attention(cache, l, 1, q_dev[l:l + 1], signs[l:l + 1], R[l:l + 1], ws, out[l:l + 1],
                                   num_splits=args.splits)
        cache.seq_len.copy_(seq0)
        one_step()                       # every kernel has run once before the capture
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            one_step()
        cache.seq_len.copy_(seq0)
        for _ in range(args.warmup):
            g.replay()
        prime()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record()
        for _ in range(args.steps):
            g.replay()
        b.record()
        barrier()
        cache.seq_len.copy_(seq0)
        return a.elapsed_time(b) / args.steps

    ms_graph = per_layer_graph_ms() if world == 1 else None
    if cache.device_status() != 0:
        raise RuntimeError("device status word set during the per-layer graph run")

    if rank != 0:
        return
    # Secondary measurements (short runs; the headline numbers above are not affected): the paper's default MXFP4
    # metadata, its captioning schedule, the prefill quantisers, and the split-K kernel on the other decode shapes.
    secondary = None
    if world == 1 and not args.no_secondary and not mx and not caption and args.workload == "step7b" and args.layers == 0:
        del cache, ws, out, in_buf, out_buf
        torch.cuda.empty_cache()
        secondary = {}
        for name, fn in (("mxfp4", lambda: quick_decode(B, dev, w, mx=True)),
                         ("caption", lambda: quick_decode(B, dev, w, caption=True)),
                         ("long7b", lambda: quick_decode(B, dev, WL.WORKLOADS["long7b"])),
                         ("step30b", lambda: quick_decode(B, dev, WL.WORKLOADS["step30b"], steps=4, warmup=2)),
                         ("prefill", lambda: run_prefill(argparse.Namespace(steps=3, warmup=1), WL.WORKLOADS["prefill7b"], B, dev, 0, emit=False)),
                         ("ladder", lambda: run_ladder(argparse.Namespace(steps=3, warmup=1), B, dev, 0, emit=False)["ladder"])):
            try:
                r = fn()
                if name == "prefill":
                    r = {k: r[k] for k in ("value", "unit", "ms_per_step", "keys_ms", "values_bulk_ms", "keys_gbs", "values_bulk_gbs",
                                           "values_bulk_tflops")} | {"frac": r["roofline"]["frac"], "workload": "prefill7b"}
                secondary[name] = r
            except Exception as e:          # a secondary number must never cost the headline line
                secondary[name] = {"error": repr(e)[:200]}
            torch.cuda.empty_cache()
    cpu = None
    if world == 1 and not args.no_cpu_baseline and not mx and not caption:
        n_l, n_s = min(4, L), min(8, Bn)
        oargs, unit_rot, th_units = oracle_prepare(w, n_l, n_s)
        passes = [oracle_pass(oargs, unit_rot) for _ in range(10)]   # ~2.5 s on 16 threads: ~40 s of CPU work
        t, threads = min(p[0] for p in passes), passes[0][1]
        cpu = {"value": th_units * BYTES_PER_TOKEN_HEAD / t / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
               "sample": f"{n_l} layers x {n_s} sequences x {H} KV heads x {N} tokens (oracle rotated-space attention, "
                         f"best of 10 passes, {t:.2f} s per pass); GB/s = packed bytes of the sample / time",
               "seconds_per_sample_pass": t}
    line = {"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "us_per_step": ms_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16-mma/f32-acc (decode), f32 (append quantisers)", "data": "synthetic",
            "config": {"workload": w.name, "n_layers": L, "batch": Bn, "n_q_heads": Hq, "n_kv_heads": H, "context": N,
                       "meta_format": args.meta, "bytes_per_token_head": bytes_th, "schedule": args.schedule,
                       "step": "okq_append(1 text token/seq, all layers) + okq_decode_attention(all layers), one call each",
                       "timed_window": f"{args.steps} consecutive steps ending on a 32-token boundary: "
                                       f"{step_kinds.get('flush_steps')} of them pack a window",
                       "decode_kernel": args.decode_kernel,
                       "packed_kv_bytes_per_step": packed_bytes, "l2": f"inputs ({packed_bytes / 1e9:.2f} GB of records per step) exceed L2",
                       "parallelism": "replicas only" if world > 1 else "1 gpu"},
            "clocks": clocks, "step_kinds": step_kinds,
            "e2e": {"value": e2e_value, "unit": "GB/s", "ms_per_step": ms_e2e / args.steps,
                    "h2d_bytes_per_step": q_host.numel() * 2 + kn_host[0].numel() * 2 + vn_host[0].numel() * 2 + Bn,
                    "d2h_bytes_per_step": out_host.numel() * 4,
                    "how": "copies on a second stream over two sets of device buffers: the transfers of neighbouring "
                           "steps overlap the kernels; timed from the first copy to the last read-back"},
            "per_layer_graph": None if ms_graph is None else {
                "us_per_step": ms_graph * 1e3, "value": packed_bytes / (ms_graph * 1e-3) / 1e9, "unit": "GB/s",
                "calls_per_step": 2 * L,
                "how": "one okq_append + one okq_decode_attention per layer, captured in one CUDA graph and replayed"},
            "gpu_launches": 3 * args.steps,
            "roofline": {"bound": "hbm", "kernel": "okq split-K decode kernel (one launch per step)",
                         "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                         "frac": achieved / peak, "frac_of_8TBs_nominal": achieved / 8000.0,
                         "kernel_ms": kernel_ms, "traffic": traffic},
            "cpu_baseline": cpu, "secondary": secondary}
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
