"""Throughput of the tensor-core prefill kernel (one layer's causal attention over a prompt).

    python -m paper_2410_18517_b200.prefill_bench [--batch B --heads Hq --kv-heads Hkv --tokens T --head-dim D --iters N]

Prints one JSON line: milliseconds per call, causal algorithmic TFLOP/s (4 B Hq D T(T+1)/2 flops: the
flops of the unmasked triangle of QK^T and PV), the tensor-core flops actually issued (the kernel runs
PV twice, for the two bf16 terms of P, and computes whole diagonal tiles), and the fraction of the
measured dense bf16 peak.  CUDA events on the launching stream, warm-up first; the K/V of a call
(>= 64 MiB at the default shape) are re-read from L2/HBM every call.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

import synth_inputs as si
from paper_2410_18517_b200 import SharedKVCache

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=2)
    ap.add_argument("--heads", type=int, default=32)
    ap.add_argument("--kv-heads", type=int, default=32)
    ap.add_argument("--tokens", type=int, default=4096)
    ap.add_argument("--head-dim", type=int, default=128, choices=[64, 128])
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args()
    B, Hq, Hkv, T, D = a.batch, a.heads, a.kv_heads, a.tokens, a.head_dim
    w = si.Workload("prefill_bench", L=2, Hq=Hq, Hkv=Hkv, D=D, B=B, context=T, dtype="bf16", n_shared=1, map_seed=0,
                    steps=1, fixed_map=(0, 0))
    cache = SharedKVCache(w.L, Hq, Hkv, D, B, T, "bf16", share_map=w.share_map())
    k, v = si.context_kv(w, 0, device="cuda")
    cache.append(0, k, v)
    q = si.normal((0, "prefill_bench_q"), (B, T, Hq, D), torch.bfloat16, device="cuda")
    out = torch.empty(B, T, Hq, D, dtype=torch.float32, device="cuda")
    layers = (0, 1)                       # layer 1 shares layer 0's slot: same bytes, other entry of the strategy
    for i in range(a.warmup):
        cache.prefill_attention(layers[i % 2], q, out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(a.iters):
        cache.prefill_attention(layers[i % 2], q, out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    algo = 4.0 * B * Hq * D * T * (T + 1) / 2
    tiles = sum(min(qb + 1, (T + 127) // 128) for qb in range((T + 127) // 128))     # 128x128 tiles visited per head
    issued = B * Hq * tiles * 3 * 2.0 * 128 * 128 * D                                 # S + PV(hi) + PV(lo)
    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops"])
        kind = "of measured"
    except Exception:
        peak, kind = 1590.0, "of fallback"
    print(json.dumps({
        "kernel": "prefill_attention_tc", "batch": B, "q_heads": Hq, "kv_heads": Hkv, "tokens": T, "head_dim": D,
        "ms_per_call": ms, "algorithmic_tflops": algo / ms / 1e9, "issued_tflops": issued / ms / 1e9,
        "roofline": {"bound": "tensor", "achieved": algo / ms / 1e9, "peak": peak, "peak_kind": kind,
                     "unit": "TFLOP/s", "frac": algo / ms / 1e9 / peak, "frac_issued": issued / ms / 1e9 / peak},
        "device_status": cache.device_status()}))


if __name__ == "__main__":
    main()
