#!/usr/bin/env python
"""Benchmark of shared-KV decode attention (KVSharer's generation path) on B200.

One *step* = one decode step of the whole model's attention path: for every layer in
order, append the new token's K/V (own-cache layers only) and run the layer's attention
over the slot the strategy points it to.  Inputs are seeded and synthetic; the cache is
resident in HBM before timing starts.

    python bench.py --gpus 1 --steps 100 --warmup 10          # this library
    python bench.py --impl reference --steps 3 --warmup 1      # the fp64 CPU oracle

The headline workload is the largest configuration that fits one GPU (`13b_mha`: 40 layers,
batch 16, context 8192 = 128K tokens per layer launch, 100 GiB of K/V read per step).  The same
JSON line carries a `configs` array with further configurations measured the same way (among them
the long-context grouped-query one and a sweep point with batch x context = 256K tokens) and a
`prefill` record for the tensor-core prefill kernel.  A timed region is exactly `--steps` decode
steps; regions are repeated (the cache cut back to the same length in between) until at least a
second has been timed, and the median region is reported.

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "shared-KV decode attention throughput (attention-path tokens/s; KV-read GB/s in roofline)"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the split-K
# kernel from the ncu captures summarised under profiles/, taken on the 4-layer cut of the
# same shape (same grid, tiles and bytes per launch).  `kv_bytes` is the algorithmic KV read
# of the captured launch; traffic grows in proportion to it, so the bench scales by that
# ratio.  A record is used only while the kernel sources still hash to `sha256`.
NCU_TRAFFIC = {
    1: {"files": ("kvs_kernels.cu", "kvs_device.cuh"), "dram_bytes": 1557.51e6, "kv_bytes": 1552.55e6,
        "sha256": "a6b6b4437657743776030cf2ad57be5b9385213ccd1d31712ac119e110e59e81"},
    2: {"files": ("kvs_mma.cu", "kvs_device.cuh"), "dram_bytes": 541.22e6, "kv_bytes": 536.90e6,
        "sha256": "e8e9a2c490fd7d0a26c8ceb3a470e7f81085cdd57c3752f23dd2b1a41da37fca"},
}


def _kernel_hash(files) -> str:
    h = hashlib.sha256()
    for f in files:
        h.update(open(os.path.join(ROOT, "paper_2410_18517_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def _peak_hbm():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi polling in a child process while the timed regions run (read-only)."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = f"/tmp/kvs_bench_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons, power = [], [], set(), []
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1])); mx.append(float(parts[2])); power.append(float(parts[3]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            # "under load": the upper half of samples by power draw
            thr = statistics.median(power)
            loaded = [s for s, p in zip(sm, power) if p >= thr] or sm
            out.update(sm_mhz=statistics.median(loaded), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power))
        return out


def cpu_sample(w):
    """Seeded inputs of 64 (sequence, q-head) units of this workload, widened to float64."""
    import torch

    n = w.context + 1
    distinct = 64
    g = torch.Generator().manual_seed(0)
    K = torch.randn(distinct, n, w.D, generator=g).to(w.torch_dtype).double().numpy()
    V = torch.randn(distinct, n, w.D, generator=g).to(w.torch_dtype).double().numpy()
    q = torch.randn(distinct, w.D, generator=g).to(w.torch_dtype).double().numpy()
    return q, K, V


def cpu_baseline(w, seconds_target: float = 15.0, sample=None) -> dict:
    """Time the oracle, as it stands, on a bounded sample of this workload's units."""
    import oracle

    q, K, V = sample if sample is not None else cpu_sample(w)
    distinct, n = K.shape[0], K.shape[1]
    oracle.attend_units(q[:8], K[:8], V[:8])            # load the library, warm the threads
    t0 = time.perf_counter()
    oracle.attend_units(q, K, V)
    t1 = time.perf_counter() - t0
    reps = max(1, min(4096, int(seconds_target / max(t1, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.attend_units(q, K, V)
    dt = time.perf_counter() - t0
    units = distinct * reps
    units_per_step = w.L * w.B * w.Hq
    step_s = dt / units * units_per_step
    return {"value": w.B / step_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{units} (sequence, q-head) units of n={n} rows ({distinct} distinct x {reps}) in {dt:.2f} s, "
                      f"extrapolated to the {units_per_step} units of one step",
            "units_per_s": units / dt}


def run_reference(args, w):
    """The oracle as the reference arm: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle

    # every step is a bounded sample; its size shrinks with the number of steps asked for so
    # that the whole run stays within about three minutes
    per_step_s = max(0.2, min(4.0, 150.0 / max(1, args.warmup + args.steps)))
    sample = cpu_sample(w)
    per = []
    for i in range(args.warmup + args.steps):
        r = cpu_baseline(w, seconds_target=per_step_s, sample=sample)
        if i >= args.warmup:
            per.append(r)
    val = statistics.mean(x["value"] for x in per)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * w.B / val, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, 1),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": per[-1]["sample"]},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def workload_config(w, n_gpus):
    return {"workload": w.name, "layers": w.L, "q_heads": w.Hq, "kv_heads": w.Hkv, "head_dim": w.D,
            "batch_per_gpu": w.B, "global_batch": w.B * n_gpus, "context": w.context,
            "batch_x_context_tokens": w.B * w.context, "storage": w.dtype,
            "shared_layers": w.n_shared, "share_map": [int(x) for x in w.share_map()],
            "parallelism": f"batch-sharded x{n_gpus}, no collective on the data path",
            "l2": "inputs larger than L2: every layer launch streams its whole slot "
                  f"({w.kv_read_bytes_per_layer(w.context) / 2**20:.0f} MiB) and "
                  f"{w.L - w.n_shared} distinct slots are cycled"}


MIN_TIMED_S = 1.0       # regions of K steps are repeated until this much has been timed (--min-seconds)
MAX_REGIONS = 200


def measure(w, K, W, E, rank, local_rank, world, dist, with_isolated=True, with_e2e=True):
    """Decode steps of workload `w` on this rank's GPU.  Returns the measurements of rank 0's line
    (every rank runs the same steps; times are the maximum over ranks)."""
    import torch

    import synth_inputs as si
    from paper_2410_18517_b200 import SharedKVCache, dist_util

    dev = torch.device("cuda", local_rank)
    sm = w.share_map()
    cache = SharedKVCache(w.L, w.Hq, w.Hkv, w.D, w.B, w.context + W + max(K, 3 + E) + 1, w.dtype, share_map=sm,
                          device=local_rank)
    # Every rank decodes its own batch of sequences (batch sharding): own seed, no exchange.
    seed = 1000 + rank
    for l in range(w.L):
        if sm[l] != l:
            continue
        k, v = si.context_kv(w, l, device=dev, base_seed=seed)
        cache.append(l, k, v)
        del k, v
    n_in = 8                                    # distinct input sets cycled over steps
    qs = [[si.step_qkv(w, t, l, device=dev, base_seed=seed) for l in range(w.L)] for t in range(n_in)]
    outs = [torch.empty(w.B, w.Hq, w.D, dtype=torch.float32, device=dev) for _ in range(w.L)]
    torch.cuda.synchronize(dev)

    def one_step(t, events=None):
        ins = qs[t % n_in]
        for l in range(w.L):
            q, k, v = ins[l]
            own = sm[l] == l
            if events is None:
                # the call a decoding loop makes: append (computing layers) + attention, the append
                # riding in the split-K kernel
                cache.decode_step(l, q, k if own else None, v if own else None, outs[l])
                continue
            if own:
                cache.append(l, k, v)
            else:
                cache.append(l, None, None, w.B, 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cache.decode_attention(l, q, outs[l])
            e1.record()
            events.append((e0, e1))

    def sync_all():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def region():
        """Exactly K steps from the same cache length, bracketed by a barrier + synchronize."""
        cache.truncate(n_start)
        sync_all()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for t in range(K):
            one_step(W + t)
        ev1.record()
        sync_all()
        return dist_util.max_over_ranks(ev0.elapsed_time(ev1), dev)

    sampler = ClockSampler(local_rank)
    for t in range(W):
        one_step(t)
    sync_all()
    n_start = cache.seq_len(0)
    if rank == 0:
        sampler.start()
        time.sleep(0.1)
    st0 = cache.stats()
    region_ms = [region()]
    st1 = cache.stats()
    # every rank derives the same count from the same (maximum-over-ranks) first region
    n_regions = max(1, min(MAX_REGIONS, int(-(-MIN_TIMED_S * 1e3 // max(region_ms[0], 1e-3)))))
    for _ in range(n_regions - 1):
        region_ms.append(region())
    clocks = sampler.stop() if rank == 0 else None
    ms = statistics.median(region_ms)
    launches = sum(st1[k] - st0[k] for k in ("append_launches", "attention_launches", "combine_launches"))
    kv_read = st1["kv_bytes_read"] - st0["kv_bytes_read"]
    kv_app = st1["kv_bytes_appended"] - st0["kv_bytes_appended"]
    n_att = st1["attention_launches"] - st0["attention_launches"]

    e2e = None
    if with_e2e:
        # End to end through the host-buffer entry point: pinned host inputs copied in, outputs copied
        # out, every step.  Same cache length as the timed regions.
        host = []
        for t in range(4):
            ql = torch.stack([qs[t][l][0] for l in range(w.L)]).cpu().pin_memory()
            kl = torch.stack([qs[t][l][1] for l in range(w.L)]).cpu().pin_memory()
            vl = torch.stack([qs[t][l][2] for l in range(w.L)]).cpu().pin_memory()
            host.append((ql, kl, vl))
        out_host = torch.empty(w.L, w.B, w.Hq, w.D, dtype=torch.float32).pin_memory()
        cache.truncate(n_start)
        for t in range(3):
            h2d, d2h = cache.step_host(*host[t % 4], out_host)
        e2e_regions = []
        for _ in range(max(1, min(n_regions, 25))):
            cache.truncate(n_start)
            sync_all()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for t in range(E):
                h2d, d2h = cache.step_host(*host[t % 4], out_host)
            e1.record()
            sync_all()
            e2e_regions.append(dist_util.max_over_ranks(e0.elapsed_time(e1), dev))
        e2e_ms = statistics.median(e2e_regions)
        e2e = {"value": dist_util.whole_job_rate(w.B, world, e2e_ms / E), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": E, "regions": len(e2e_regions), "ms_per_step": e2e_ms / E,
               "context_mid_run": n_start + E // 2,
               "how": "kvs_step_host: pinned host q/k/v in, fp32 outputs back to pinned host memory, every step"}

    isolated = None
    if with_isolated:
        # The same K steps with a CUDA event pair around every attention call: the duration of the
        # dominant kernel's launches (split-K kernel + its small combine) with the overlap forbidden.
        cache.truncate(n_start)
        events = []
        rb0 = cache.stats()["kv_bytes_read"]
        for t in range(K):
            one_step(W + t, events)
        sync_all()
        att_ms = [a.elapsed_time(b) for a, b in events]
        att_bytes = cache.stats()["kv_bytes_read"] - rb0
        isolated = (sum(att_ms) / len(att_ms), att_bytes / len(att_ms), len(att_ms))

    status = cache.device_status()
    rec = None
    if rank == 0:
        peak, peak_kind = _peak_hbm()
        # Dominant kernel = the split-K attention kernel, one launch per layer.  Its average launch
        # duration over the timed region is the region's CUDA-event time divided by its launches: the
        # kernels of a step overlap (early-start launches), so this includes the hidden remainders of
        # the combine kernels and is a lower bound on the kernel's own rate.
        pipelined_ms = ms / n_att
        pipelined_bytes = kv_read / n_att
        achieved = pipelined_bytes / (pipelined_ms * 1e-3) / 1e9
        traffic = None
        kernel_id = cache.last_launch()["kernel"]
        nrec = NCU_TRAFFIC.get(kernel_id)
        if nrec and nrec["sha256"] == _kernel_hash(nrec["files"]):
            traffic = nrec["dram_bytes"] * pipelined_bytes / nrec["kv_bytes"]
        step_ms = ms / K
        pool_unshared = cache.pool_bytes // cache.num_slots() * w.L
        roofline = {"bound": "hbm", "kernel": ("decode_splitk_scalar", "decode_splitk_mma")[kernel_id - 1]
                    + " (timed region / launches; the append rides in it, the combine kernel overlaps it)",
                    "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                    "frac": achieved / peak, "frac_of_8tbs_nominal": achieved / NOMINAL_HBM_GBS,
                    "traffic": traffic, "bytes_per_launch": pipelined_bytes, "ms_per_launch": pipelined_ms,
                    "launches_timed": n_att, "ctas": cache.last_launch()["ctas"]}
        if isolated is not None:
            iso = isolated[1] / (isolated[0] * 1e-3) / 1e9
            roofline["isolated"] = {"achieved": iso, "frac": iso / peak, "ms_per_call": isolated[0],
                                    "bytes_per_launch": isolated[1], "launches_timed": isolated[2],
                                    "how": "event pair around every attention call (split-K + combine), no overlap"}
        rec = {
            "value": dist_util.whole_job_rate(w.B, world, step_ms), "unit": UNIT, "ms_per_step": step_ms,
            "config": workload_config(w, world),
            "timed": {"regions": len(region_ms), "steps_per_region": K, "seconds": sum(region_ms) * 1e-3,
                      "region_ms_min": min(region_ms), "region_ms_median": ms, "region_ms_max": max(region_ms),
                      "how": "each region is exactly `steps` decode steps from the same cache length (kvs_truncate "
                             "in between), barrier + synchronize on both sides, CUDA events, max over ranks; the "
                             "median region is reported"},
            "kv_read_gbs_whole_step": kv_read / (ms * 1e-3) / 1e9,
            "kv_read_frac_of_8tbs_nominal": kv_read / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            "kv_bytes_read_per_step": kv_read // K, "kv_bytes_appended_per_step": kv_app // K,
            "pool_bytes": cache.pool_bytes, "pool_bytes_unshared": pool_unshared,
            "kv_memory_saved_frac": 1.0 - cache.pool_bytes / pool_unshared,
            "context_mid_run": n_start + K // 2,
            "roofline": roofline, "e2e": e2e, "gpu_launches": launches, "clocks": clocks, "device_status": status,
            "ms_per_step_x_sm_mhz": step_ms * clocks["sm_mhz"] if clocks and clocks.get("sm_mhz") else None,
        }
    cache.close()
    del cache, qs, outs
    import gc

    gc.collect()
    torch.cuda.empty_cache()
    return rec


def search_record(local_rank):
    """The strategy search's reductions (layer-pair KV distances on the paper's calibration shape for a 7B and a
    13B model, the mean-representation cosine on 1 GB) and decode over an evicted slot: time and GB/s of
    algorithmic bytes against the measured copy bandwidth."""
    import torch

    from paper_2410_18517_b200 import next_rows_bench as nr

    peak, kind = _peak_hbm()
    out = []
    with torch.cuda.device(local_rank):
        for rec in (nr.distances(32, 32, 30, 64), nr.distances(40, 40, 30, 64), nr.cosine(30, 2048 * 4096),
                    nr.ragged_decode(32, 8, 4, 32768, 0.8)):
            gbs = rec.get("gbs", rec.get("kv_gbs_of_existing_rows"))
            rec["roofline"] = {"bound": "hbm", "achieved": gbs, "peak": peak, "peak_kind": f"of {kind}", "unit": "GB/s",
                               "frac": gbs / peak}
            out.append(rec)
    return out


def prefill_record(local_rank):
    """The tensor-core prefill kernel on two prompt shapes: ms per call and TFLOP/s against the
    measured dense bf16 peak (algorithmic = causal flops 4 B Hq D T(T+1)/2; issued = what the tensor
    cores are given: S plus two PV terms over whole tiles)."""
    import torch

    import synth_inputs as si
    from paper_2410_18517_b200 import SharedKVCache

    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops"])
        kind = "of measured"
    except Exception:
        peak, kind = 1590.0, "of fallback"
    out = []
    for (B, Hq, Hkv, T) in ((2, 32, 32, 4096), (1, 32, 8, 16384)):
        D = 128
        w = si.Workload("prefill_bench", L=2, Hq=Hq, Hkv=Hkv, D=D, B=B, context=T, dtype="bf16", n_shared=1,
                        map_seed=0, steps=1, fixed_map=(0, 0))
        cache = SharedKVCache(w.L, Hq, Hkv, D, B, T, "bf16", share_map=w.share_map(), device=local_rank)
        dev = cache.device
        k, v = si.context_kv(w, 0, device=dev)
        cache.append(0, k, v)
        q = si.normal((0, "prefill_bench_q"), (B, T, Hq, D), torch.bfloat16, device=dev)
        o = torch.empty(B, T, Hq, D, dtype=torch.float32, device=dev)
        for i in range(3):
            cache.prefill_attention(i % 2, q, o)
        torch.cuda.synchronize(dev)
        iters = 20
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            cache.prefill_attention(i % 2, q, o)     # layer 1 shares layer 0's slot
        e1.record()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1) / iters
        algo = 4.0 * B * Hq * D * T * (T + 1) / 2
        tiles = sum(min(qb + 1, (T + 127) // 128) for qb in range((T + 127) // 128))
        issued = B * Hq * tiles * 3 * 2.0 * 128 * 128 * D
        out.append({"kernel": "prefill_attention_tc", "batch": B, "q_heads": Hq, "kv_heads": Hkv, "tokens": T,
                    "head_dim": D, "ms_per_call": ms, "algorithmic_tflops": algo / ms / 1e9,
                    "issued_tflops": issued / ms / 1e9,
                    "roofline": {"bound": "tensor", "achieved": algo / ms / 1e9, "peak": peak, "peak_kind": kind,
                                 "unit": "TFLOP/s", "frac": algo / ms / 1e9 / peak,
                                 "frac_issued": issued / ms / 1e9 / peak},
                    "device_status": cache.device_status()})
        cache.close()
        del cache, k, v, q, o
        torch.cuda.empty_cache()
    return out


DEFAULT_WORKLOAD = "13b_mha"
DEFAULT_CONFIGS = "gqa_long,sweep_b32_n8192_p10,7b_mha"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="kvs", choices=["kvs", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--configs", default=None,
                    help="comma-separated further configurations for the `configs` array ('' = none; default: "
                         f"{DEFAULT_CONFIGS} when the headline workload is the default one, at 1 GPU)")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true")
    ap.add_argument("--no-search", action="store_true", help="skip the record of the search reductions and the evicted-slot decode")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_S,
                    help="regions of --steps steps are repeated until this much has been timed (0: one region, for "
                         "profiler captures)")
    args = ap.parse_args()
    globals()["MIN_TIMED_S"] = args.min_seconds
    if args.warmup < 3 and args.impl == "kvs":
        args.warmup = 3

    import synth_inputs as si

    w = si.workload_by_name(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch

    from paper_2410_18517_b200 import build as kbuild

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist

        if rank == 0:
            kbuild.build()
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        kbuild.build()
    torch.cuda.set_device(local_rank)
    if dist is not None:
        dist.barrier()

    K, W, E = args.steps, args.warmup, args.e2e_steps
    head = measure(w, K, W, E, rank, local_rank, world, dist)
    extras, prefill, search = [], None, None
    if world == 1:
        names = args.configs if args.configs is not None else (DEFAULT_CONFIGS if args.workload == DEFAULT_WORKLOAD else "")
        for name in [x for x in names.split(",") if x]:
            r = measure(si.workload_by_name(name), K, W, E, rank, local_rank, world, dist, with_isolated=False,
                        with_e2e=False)
            r.pop("e2e", None)
            extras.append(r)
        if not args.no_prefill:
            prefill = prefill_record(local_rank)
        if not args.no_search and args.workload == DEFAULT_WORKLOAD and args.configs is None:   # the full default run only
            search = search_record(local_rank)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    line = {"metric": METRIC, "value": head.pop("value"), "unit": head.pop("unit"), "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": head.pop("ms_per_step"), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic"}
    line.update(head)
    if extras:
        line["configs"] = extras
    if prefill is not None:
        line["prefill"] = prefill
    if search is not None:
        line["search_and_evicted"] = search
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
