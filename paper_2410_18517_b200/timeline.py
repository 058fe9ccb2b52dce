"""Per-block timeline of the decode-attention kernels, from the tracing build of the library.

    python -m paper_2410_18517_b200.timeline [--batch B --context N --heads Hq --kv-heads Hkv --layers L --steps S]

Builds ``libkvs_trace.so`` (the library compiled with -DKVS_TRACE), runs a few decode steps
(``kvs_decode_step`` per layer, launched call by call) and prints, for the launches of the last steps, when
the thread blocks of the split-K kernel entered, when their wait for the previous kernel returned, when
their first tile arrived, when their pieces and the blocks themselves ended, and when the combine kernel
(if the call needs one) waited and ended: all in microseconds after the launch's first block entered, as
minimum / median / maximum over the blocks, medians over the launches.  Stamps are the GPU's nanosecond
timer (its resolution here is about a quarter of a microsecond).
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

import synth_inputs as si
from paper_2410_18517_b200 import SharedKVCache, binding
from paper_2410_18517_b200 import build as kbuild

binding.LIB_PATH = kbuild.LIB_TRACE          # this process works with the tracing build (nothing is loaded yet)

ROWS, SLOTS = 160, 32


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--context", type=int, default=1024)
    ap.add_argument("--heads", type=int, default=32)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--steps", type=int, default=3, help="traced steps (after 4 untraced ones); the first traced step is not reported")
    a = ap.parse_args()
    kbuild.build(trace=True)
    w = si.Workload(f"timeline_b{a.batch}_n{a.context}", L=a.layers, Hq=a.heads, Hkv=a.kv_heads, D=128, B=a.batch,
                    context=a.context, dtype="bf16", n_shared=a.layers // 4, map_seed=1, steps=a.steps)
    dev = torch.device("cuda", 0)
    sm = w.share_map()
    cache = SharedKVCache(w.L, w.Hq, w.Hkv, w.D, w.B, w.context + 64, w.dtype, share_map=sm)
    k, v = si.context_kv(w, 0, device=dev)
    for l in range(w.L):
        if sm[l] == l:
            cache.append(l, k, v)
    ins = [si.step_qkv(w, 0, l, device=dev) for l in range(w.L)]
    outs = [torch.empty(w.B, w.Hq, w.D, dtype=torch.float32, device=dev) for _ in range(w.L)]

    def one_step():
        for l in range(w.L):
            q, kk, vv = ins[l]
            own = sm[l] == l
            cache.decode_step(l, q, kk if own else None, vv if own else None, outs[l])

    for _ in range(4):
        one_step()
    torch.cuda.synchronize()
    n_launches = a.steps * w.L
    buf = torch.zeros(n_launches * ROWS * SLOTS, dtype=torch.int64, device=dev)
    binding.kvs_trace_begin(cache.ctx, buf, buf.numel() * 8)
    for _ in range(a.steps):
        one_step()
    torch.cuda.synchronize()
    recorded = binding.kvs_trace_end(cache.ctx)
    assert recorded == n_launches and cache.device_status() == 0
    t = buf.cpu().numpy().reshape(n_launches, ROWS, SLOTS).astype(np.float64)
    ctas = cache.last_launch()["ctas"]

    def mmm(x):
        return [float(x.min()), float(np.median(x)), float(x.max())]

    per = []
    prev_base = None
    for li in range(w.L, n_launches):                  # the first traced step is warm-up for the stamps' caches
        blk = t[li, :ctas]
        base = blk[:, 0].min()
        us = lambda col: mmm((blk[:, col] - base) / 1e3)          # noqa: E731
        rec = {"entry": us(0), "producer_wait_returns": us(1), "consumer_wait_returns": us(2), "first_tile": us(3),
               "end": us(20)}
        pieces = blk[:, 21].astype(int)
        rec["pieces_per_block"] = float(pieces.mean())
        merges = [blk[pieces > kk, 5 + 2 * kk] - blk[pieces > kk, 4 + 2 * kk] for kk in range(8) if (pieces > kk).any()]
        rec["piece_merge_us"] = float(np.median(np.concatenate(merges)) / 1e3)
        rec["stream_us_median_block"] = float(np.median(blk[:, 20] - blk[:, 3]) / 1e3)
        c0, c1 = t[li, 150], t[li, 151]
        if c0[2] > 0:
            rec["combine_first_block"] = [float((c0[i] - base) / 1e3) for i in range(3)]
            rec["combine_last_block"] = [float((c1[i] - base) / 1e3) for i in range(3)]
        if prev_base is not None:
            rec["period"] = float((base - prev_base) / 1e3)
        prev_base = base
        per.append(rec)
    # Is a block late because of the SM it ran on?  Per launch: each block's stream time (first tile to end)
    # relative to the launch's median; then, per SM, the mean over the launches (what is systematic) and the
    # spread of the rest (what is not).
    rel, sms = [], []
    for li in range(w.L, n_launches):
        blk = t[li, :ctas]
        d = blk[:, 20] - blk[:, 3]
        rel.append(d / np.median(d) - 1.0)
        sms.append(blk[:, 23].astype(int))
    rel, sms = np.concatenate(rel), np.concatenate(sms)
    per_sm = {int(sm_): rel[sms == sm_] for sm_ in np.unique(sms)}
    sm_mean = np.array([v.mean() for v in per_sm.values()])
    resid = np.concatenate([v - v.mean() for v in per_sm.values()])
    out_sm = {"sms_seen": len(per_sm), "systematic_std_pct": round(100 * float(sm_mean.std()), 2),
              "systematic_min_max_pct": [round(100 * float(sm_mean.min()), 2), round(100 * float(sm_mean.max()), 2)],
              "residual_std_pct": round(100 * float(resid.std()), 2)}
    out = {"workload": {"batch": a.batch, "context": a.context, "q_heads": a.heads, "kv_heads": a.kv_heads, "layers": a.layers,
                        "kernel": cache.last_launch()["kernel"], "blocks": ctas,
                        "kv_mb_per_launch": w.kv_read_bytes_per_layer(w.context) / 1e6,
                        "combine_launches": cache.stats()["combine_launches"]},
           "launches_reported": len(per), "stream_time_by_sm": out_sm}
    for key in ("entry", "producer_wait_returns", "consumer_wait_returns", "first_tile", "end", "combine_first_block",
                "combine_last_block"):
        vals = [r[key] for r in per if key in r]
        if vals:
            out[key] = [round(float(np.median([v[i] for v in vals])), 2) for i in range(3)]
    for key in ("pieces_per_block", "piece_merge_us", "stream_us_median_block", "period"):
        vals = [r[key] for r in per if key in r]
        out[key] = round(float(np.median(vals)), 2)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
