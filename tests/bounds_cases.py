"""Cases run against the bounds-checking build of the library (-DKVS_DEBUG_BOUNDS).

Run as a script by tests/test_gpu_bounds.py with KVS_LIBRARY pointing at libkvs_bounds.so.  In that
build every global offset the kernels compute is checked on the device; a violation sets the device
status word to KVS_ERR_BOUNDS.  On top of that the pool sits between guard zones and every row no
token may occupy carries a pattern (helpers.GuardedCache).  Each case must match the oracle as in
the normal build, end with a clean status word and leave every canary untouched.
"""
import sys

import numpy as np
import torch

import helpers
import oracle
import synth_inputs as si
from paper_2410_18517_b200 import KVS_OPT_KERNEL, KVS_OPT_REPLAY
from paper_2410_18517_b200 import binding as kb

helpers.CACHE_CLASS = helpers.GuardedCache


def tiny_whole():
    cache, _, _ = helpers.run_small(si.WORKLOADS["tiny"], steps=9)
    cache.check_canaries()


def decode_steps():
    for (dtype, D, Hq, Hkv, B, kernel) in (("bf16", 128, 4, 4, 3, 1), ("bf16", 128, 8, 2, 3, 2), ("bf16", 64, 8, 2, 2, 2),
                                           ("f32", 128, 4, 2, 2, 1), ("bf16", 128, 8, 8, 24, 0), ("bf16", 128, 16, 4, 40, 0)):
        for context in (0, 63, 127, 700):
            w = si.Workload(f"b_{dtype}_{D}_{Hq}_{Hkv}_{B}_{context}", L=3, Hq=Hq, Hkv=Hkv, D=D, B=B, context=context,
                            dtype=dtype, n_shared=1, map_seed=0, steps=3, fixed_map=(0, 1, 0))
            opts = [(KVS_OPT_KERNEL, kernel)] if kernel else []
            for use_step in (False, True):
                cache, _, _ = helpers.run_small(w, steps=3, options=opts, use_step=use_step)
                cache.check_canaries()


def smaller_batch_than_capacity():
    """max_batch above the batch in use: whole units of every plane are canaries."""
    w = si.Workload("b_small_batch", L=2, Hq=8, Hkv=2, D=128, B=3, context=300, dtype="bf16", n_shared=1, map_seed=0,
                    steps=2, fixed_map=(0, 0))
    sm = w.share_map()
    cache = helpers.make_cache(w, 5, sm, max_batch=5)
    orc = oracle.Oracle(w.L, w.Hq, w.Hkv, w.D, w.B, sm)
    k, v = si.context_kv(w, 0)
    orc.layer_forward(0, None, k.double().numpy(), v.double().numpy())
    cache.append(0, k.cuda(), v.cuda())
    for t in range(4):
        for l in range(w.L):
            q, k, v = si.step_qkv(w, t, l)
            ref = orc.layer_forward(l, q.double().numpy(), k.double().numpy(), v.double().numpy())
            out = cache.decode_step(l, q.cuda(), k.cuda() if l == 0 else None, v.cuda() if l == 0 else None)
            helpers.assert_close(out.cpu().numpy(), ref, f"small batch step {t} layer {l}")
    assert cache.device_status() == 0
    cache.check_canaries()


def ragged():
    w = si.Workload("b_ragged", L=2, Hq=8, Hkv=2, D=128, B=2, context=333, dtype="bf16", n_shared=1, map_seed=0, steps=3,
                    fixed_map=(0, 0))
    sm = w.share_map()
    cache = helpers.make_cache(w, 4, sm)
    orc = oracle.Oracle(w.L, w.Hq, w.Hkv, w.D, w.B, sm)
    k, v = si.context_kv(w, 0)
    orc.layer_forward(0, None, k.double().numpy(), v.double().numpy())
    cache.append(0, k.cuda(), v.cuda())
    rng = np.random.default_rng(5)
    n_keep = rng.integers(40, 333, size=(w.B, w.Hkv)).astype(np.int32)
    keep = np.zeros((w.B, w.Hkv, 333), dtype=np.int32)
    for b in range(w.B):
        for h in range(w.Hkv):
            keep[b, h, : n_keep[b, h]] = np.sort(rng.choice(333, size=n_keep[b, h], replace=False))
    cache.evict(0, torch.from_numpy(keep).cuda(), n_keep)
    orc.evict(0, keep, n_keep)
    for t in range(3):
        for l in range(w.L):
            q, k, v = si.step_qkv(w, t, l)
            ref = orc.layer_forward(l, q.double().numpy(), k.double().numpy(), v.double().numpy())
            out = cache.decode_step(l, q.cuda(), k.cuda() if l == 0 else None, v.cuda() if l == 0 else None)
            helpers.assert_close(out.cpu().numpy(), ref, f"ragged step {t} layer {l}")
    assert cache.device_status() == 0
    cache.check_canaries()


def replay_past_capacity():
    """A recorded step replayed beyond max_seq appends nothing more and reports CAPACITY, not a stray write."""
    for (Hq, Hkv, use_step) in ((4, 4, False), (8, 2, True)):
        w = si.Workload(f"b_replay_{Hq}_{Hkv}", L=2, Hq=Hq, Hkv=Hkv, D=128, B=2, context=250, dtype="bf16", n_shared=1,
                        map_seed=0, steps=1, fixed_map=(0, 0))
        cache = helpers.make_cache(w, 4)              # room for four more tokens only
        cache.set_option(KVS_OPT_REPLAY, 1)
        k, v = si.context_kv(w, 0, device="cuda")
        cache.append(0, k, v)
        q, kk, vv = si.step_qkv(w, 0, 0, device="cuda")
        outs = [torch.empty(w.B, w.Hq, w.D, dtype=torch.float32, device="cuda") for _ in range(w.L)]

        def step():
            for l in range(w.L):
                if use_step:
                    cache.decode_step(l, q, kk if l == 0 else None, vv if l == 0 else None, outs[l])
                else:
                    cache.append(l, kk if l == 0 else None, vv if l == 0 else None, w.B, 1)
                    cache.decode_attention(l, q, outs[l])
            cache.replay_advance()

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()                                    # eager: token 251
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                step()                                # recorded as token 252
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(6):                            # tokens 252 .. 254 fit, the rest do not
            g.replay()
        torch.cuda.synchronize()
        assert cache.device_status() == kb.KVS_ERR_CAPACITY
        assert all(bool(torch.isfinite(o).all()) for o in outs)
        cache.check_canaries()


def prefill():
    w = si.Workload("b_prefill", L=2, Hq=4, Hkv=2, D=128, B=2, context=300, dtype="bf16", n_shared=1, map_seed=0, steps=1,
                    fixed_map=(0, 0))
    sm = w.share_map()
    cache = helpers.make_cache(w, 0, sm)
    orc = oracle.Oracle(w.L, w.Hq, w.Hkv, w.D, w.B, sm)
    k, v = si.context_kv(w, 0)
    cache.append(0, k.cuda(), v.cuda())
    for l in range(w.L):
        q = si.normal((0, "b_prefill_q", l), (w.B, w.context, w.Hq, w.D), torch.bfloat16)
        ref = orc.layer_prefill(l, q.double().numpy(), k.double().numpy() if l == 0 else None,
                                v.double().numpy() if l == 0 else None)
        out = cache.prefill_attention(l, q.cuda())
        helpers.assert_close(out.cpu().numpy(), ref, f"prefill layer {l}")
    assert cache.device_status() == 0
    cache.check_canaries()


def the_check_itself_records_a_violation():
    """An offset outside its buffer, handed to the check without any memory access: status 9."""
    w = si.WORKLOADS["tiny"]
    cache = helpers.make_cache(w, 2)
    assert cache.device_status() == 0
    kb.kvs_selftest_bounds(cache.ctx, torch.cuda.current_stream().cuda_stream)
    assert cache.device_status() == kb.KVS_ERR_BOUNDS
    cache.clear_device_status()
    assert cache.device_status() == 0
    cache.check_canaries()


if __name__ == "__main__":
    assert kb.LIB_PATH.endswith("libkvs_bounds.so"), kb.LIB_PATH
    for case in (the_check_itself_records_a_violation, tiny_whole, decode_steps, smaller_batch_than_capacity, ragged, replay_past_capacity, prefill):
        case()
        print("ok", case.__name__, flush=True)
    print("ALL BOUNDS CASES PASSED")
