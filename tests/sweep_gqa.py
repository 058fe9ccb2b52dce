"""Sweep of the grouped-query shape (32 layers, 32 q-heads / 8 kv-heads, D=128, bf16) over batch,
context and shared-layer fraction.  One JSON line per point: parity of sampled units with the fp64
oracle, time per decode step, attention-path tokens/s, KV-read GB/s and pool size.

    python tests/sweep_gqa.py [--out FILE] [--steps K] [--only B,N,P] [--shared P] [--kernel K] [--samples S]

A *step* is one pass over all layers (kvs_decode_step per layer: append on computing layers, riding in
the attention kernel, + attention on every layer).
--kernel forces KVS_OPT_KERNEL (1 scalar, 2 tensor-core) instead of the library's own choice.
Each point is timed twice: launched call by call from Python, and as replays of a CUDA graph of one
recorded step (which takes the host's launch cost out; with the library's replay counter every
replay is the next decode step, one row further along).
Before a point is timed, every computing layer is loaded with its own seeded context and one decode
step is compared with the oracle on sampled (layer, sequence, q-head) units (every sharing layer is
among them); the worst errors go into the point's record, and a point outside the tolerance stops
the sweep.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
for p in (ROOT, os.path.join(ROOT, "tests")):
    if p not in sys.path:
        sys.path.insert(0, p)

import synth_inputs as si  # noqa: E402
from helpers import SampledRun  # noqa: E402
from paper_2410_18517_b200 import KVS_OPT_KERNEL, KVS_OPT_REPLAY  # noqa: E402

HBM_BYTES_USABLE = 170 * 2**30      # leave head-room below the 180 GB of a B200


def pool_bytes(w: si.Workload, extra_rows: int) -> int:
    rs = (w.context + extra_rows + 127) // 128 * 128
    return (w.L - w.n_shared) * 2 * w.B * w.Hkv * rs * w.D * w.elem_bytes


def time_point(w: si.Workload, steps: int, device=0, kernel=0, samples=8) -> dict:
    extra = 3 * steps + 24
    rec = {"workload": w.name, "batch": w.B, "context": w.context, "shared_layers": w.n_shared,
           "pool_bytes": pool_bytes(w, extra), "pool_bytes_unshared": pool_bytes(w.scaled(n_shared=0), extra)}
    if rec["pool_bytes"] > HBM_BYTES_USABLE:
        rec["fits"] = False
        return rec
    rec["fits"] = True
    sm = w.share_map()
    rec["share_map"] = [int(x) for x in sm]
    dev = torch.device("cuda", device)
    # parity first: own seeded context per computing layer, one decode step against the oracle on
    # sampled units (the sharing layers plus random ones), the cached rows of those units bit for bit
    run = SampledRun(w, extra, n_samples=w.n_shared + samples, seed=1, device=device)
    cache = run.cache
    if kernel:
        cache.set_option(KVS_OPT_KERNEL, kernel)
    run.load_context()
    worst = run.step(0, check=True)
    run.check_cached_rows()
    rec.update(parity_units=len(run.samples), parity_max_abs=worst[0], parity_rel_l2=worst[1])
    ins = [si.step_qkv(w, 0, l, device=dev) for l in range(w.L)]
    outs = [torch.empty(w.B, w.Hq, w.D, dtype=torch.float32, device=dev) for _ in range(w.L)]

    def one_step(replay=False):
        for l in range(w.L):
            q, kk, vv = ins[l]
            own = sm[l] == l
            cache.decode_step(l, q, kk if own else None, vv if own else None, outs[l])
        if replay:
            cache.replay_advance()       # recorded only while capturing

    def timed(fn, n):
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / n

    for _ in range(3):
        one_step()
    b0 = cache.stats()["kv_bytes_read"]
    ms = timed(one_step, steps)
    read_per_step = (cache.stats()["kv_bytes_read"] - b0) / steps
    rec.update(ms_per_step=ms, tokens_per_s=w.B / (ms * 1e-3), kv_read_gbs=read_per_step / (ms * 1e-3) / 1e9,
               kv_bytes_read_per_step=read_per_step, kernel=cache.last_launch()["kernel"],
               ctas=cache.last_launch()["ctas"])

    # graph replays of one recorded step; the replay counter makes every replay the next step
    cache.set_option(KVS_OPT_REPLAY, 1)
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream(dev))
    with torch.cuda.stream(side):
        one_step(True)
        graph = torch.cuda.CUDAGraph()
        b0 = cache.stats()["kv_bytes_read"]
        with torch.cuda.graph(graph, stream=side):
            one_step(True)
        read_graph = cache.stats()["kv_bytes_read"] - b0
    torch.cuda.current_stream(dev).wait_stream(side)
    graph.replay()
    ms_g = timed(graph.replay, steps)
    cache.replay_commit(1 + steps)
    torch.cuda.synchronize(dev)
    rec.update(replayed_to=cache.seq_len(0))
    rec.update(graph_ms_per_step=ms_g, graph_tokens_per_s=w.B / (ms_g * 1e-3),
               graph_kv_read_gbs=read_graph / (ms_g * 1e-3) / 1e9, device_status=cache.device_status())
    cache.close()
    del cache, run, ins, outs, graph
    torch.cuda.empty_cache()
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--only", default=None, help="B,N,P of a single point")
    ap.add_argument("--shared", type=int, default=None, help="only the points with this many shared layers")
    ap.add_argument("--kernel", type=int, default=0, help="force KVS_OPT_KERNEL (0 = the library's choice)")
    ap.add_argument("--samples", type=int, default=8, help="sampled units beyond the sharing layers checked per point")
    args = ap.parse_args()
    pts = si.sweep_points()
    if args.shared is not None:
        pts = [p for p in pts if p.n_shared == args.shared]
    if args.only:
        B, N, P = (int(x) for x in args.only.split(","))
        pts = [p for p in pts if (p.B, p.context, p.n_shared) == (B, N, P)]
    f = open(args.out, "w") if args.out else None
    for w in pts:
        rec = time_point(w, args.steps, kernel=args.kernel, samples=args.samples)
        line = json.dumps(rec)
        print(line, flush=True)
        if f:
            f.write(line + "\n")
            f.flush()
    if f:
        f.close()


if __name__ == "__main__":
    sys.exit(main())
