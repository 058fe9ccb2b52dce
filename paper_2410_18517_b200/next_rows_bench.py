"""Timings of the widened rows: decode over evicted (ragged) slots and the strategy-search reductions.

    python -m paper_2410_18517_b200.next_rows_bench

One JSON line per measurement (CUDA events, warm-up first, no profiler).  GB/s figures are
algorithmic bytes (rows that exist x row bytes, read once) over time.
"""
from __future__ import annotations

import json

import numpy as np
import torch

import synth_inputs as si
from paper_2410_18517_b200 import SharedKVCache


def timed(fn, iters=20, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def ragged_decode(Hq, Hkv, B, n, keep_frac, slots=4):
    """Attention over slots from which an outside method evicted (1 - keep_frac) of the rows at random."""
    w = si.Workload("ragged_bench", L=slots, Hq=Hq, Hkv=Hkv, D=128, B=B, context=n, dtype="bf16", n_shared=0,
                    map_seed=0, steps=1)
    cache = SharedKVCache(slots, Hq, Hkv, 128, B, n + 8, "bf16")
    rng = np.random.default_rng(0)
    rows = 0
    for l in range(slots):
        k, v = si.context_kv(w, l, device="cuda")
        cache.append(l, k, v)
        del k, v
        if keep_frac < 1.0:
            n_keep = rng.binomial(n, keep_frac, size=(B, Hkv)).clip(1, n).astype(np.int32)
            keep = np.zeros((B, Hkv, n), dtype=np.int32)
            for b in range(B):
                for h in range(Hkv):
                    keep[b, h, : n_keep[b, h]] = np.sort(rng.choice(n, size=n_keep[b, h], replace=False))
            cache.evict(l, torch.from_numpy(keep).cuda(), n_keep)
            rows += int(n_keep.sum())
        else:
            rows += B * Hkv * n
    q = si.step_qkv(w, 0, 0, device="cuda")[0]
    out = torch.empty(B, Hq, 128, dtype=torch.float32, device="cuda")
    i = [0]

    def f():
        cache.decode_attention(i[0] % slots, q, out)
        i[0] += 1
    ms = timed(f, iters=5 * slots)
    by = 2.0 * rows / slots * 256
    rec = {"what": "decode over evicted slots", "q_heads": Hq, "kv_heads": Hkv, "batch": B, "rows_before": n,
           "kept_fraction": keep_frac, "us_per_call": ms * 1e3, "kv_gbs_of_existing_rows": by / ms / 1e6,
           "device_status": cache.device_status()}
    cache.close()
    return rec


def distances(L, Hkv, B, n, D=128):
    w = si.Workload("dist_bench", L=L, Hq=Hkv, Hkv=Hkv, D=D, B=B, context=n, dtype="bf16", n_shared=0, map_seed=0, steps=0)
    cache = SharedKVCache(L, Hkv, Hkv, D, B, n, "bf16")
    k, v = si.context_kv(w, 0, device="cuda")
    for l in range(L):
        cache.append(l, torch.roll(k, l, 1), v)
    ms = timed(lambda: cache.layer_distances(B), iters=10)
    by = 2.0 * L * B * Hkv * n * D * 2
    rec = {"what": "layer-pair KV distances", "layers": L, "samples": B, "tokens": n, "kv_heads": Hkv, "head_dim": D,
           "ms_per_call": ms, "bytes_read": by, "gbs": by / ms / 1e6, "device_status": cache.device_status()}
    cache.close()
    return rec


def cosine(S, dim):
    cache = SharedKVCache(1, 1, 1, 64, 1, 8, "bf16")
    a = torch.randn(S, dim, device="cuda").bfloat16()
    b = torch.randn(S, dim, device="cuda").bfloat16()
    ms = timed(lambda: cache.mean_cosine(a, b), iters=10)
    by = 2.0 * S * dim * 2
    return {"what": "mean-representation cosine", "samples": S, "dim": dim, "us_per_call": ms * 1e3,
            "bytes_read": by, "gbs": by / ms / 1e6}


def main():
    for rec in (ragged_decode(32, 32, 8, 4096, 1.0), ragged_decode(32, 32, 8, 4096, 0.8),
                ragged_decode(32, 8, 4, 32768, 0.8), ragged_decode(32, 8, 4, 32768, 0.5),
                distances(32, 32, 30, 64), distances(40, 40, 30, 64), distances(32, 8, 30, 2048),
                cosine(30, 64 * 4096), cosine(30, 2048 * 4096)):
        print(json.dumps(rec), flush=True)


if __name__ == "__main__":
    main()
