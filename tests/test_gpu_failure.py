"""Failure detection on the device: the give-up path of the bounded waits.

Every wait inside the pipelined kernels is bounded.  Nothing in the normal tests ever makes one
run out, so this file makes one run out on purpose, in the harmless way: a one-warp self-test kernel
waits, with a limit of about a millisecond, on a barrier that nothing arrives at (no copy is in
flight, nothing traps), through the very function the attention kernels wait with.  The wait gives
up, the status word reads KVS_ERR_TIMEOUT, the kernel returns, and the context goes on working.
"""
import os

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_2410_18517_b200 import KvsError, SharedKVCache
from paper_2410_18517_b200 import binding as kb
from paper_2410_18517_b200 import build as kbuild

from helpers import assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


def _small_cache():
    w = si.Workload("failure_case", L=2, Hq=4, Hkv=2, D=128, B=2, context=300, dtype="bf16", n_shared=1, map_seed=0,
                    steps=1, fixed_map=(0, 0))
    cache = SharedKVCache(w.L, w.Hq, w.Hkv, w.D, w.B, w.context + 4, w.dtype, share_map=w.share_map())
    k, v = si.context_kv(w, 0)
    cache.append(0, k.cuda(), v.cuda())
    return w, cache, k, v


@pytest.mark.parametrize("limit_us", [200, 1000, 5000])
def test_a_wait_that_nothing_ends_runs_out_and_reports(limit_us):
    w, cache, k, v = _small_cache()
    assert cache.device_status() == 0
    waited_ns = cache.selftest_wait_timeout(limit_us)
    assert cache.device_status() == kb.KVS_ERR_TIMEOUT
    # the wait lasted about as long as it was allowed to: not cut short, not far over
    assert limit_us * 1000 <= waited_ns <= limit_us * 1000 + 2_000_000, waited_ns
    # the context is intact: clear the word, run a normal call, compare with the oracle
    cache.clear_device_status()
    assert cache.device_status() == 0
    q = si.step_qkv(w, 0, 1)[0]
    out = cache.decode_attention(1, q.cuda()).cpu().numpy()
    K, V = k.double().numpy(), v.double().numpy()
    for b in range(w.B):
        for hq in range(w.Hq):
            ref = oracle.attend_unit(q[b, hq].double().numpy(), K[b, :, hq // w.G], V[b, :, hq // w.G])
            assert_close(out[b, hq], ref, f"after the self-test, unit {(b, hq)}")
    assert cache.device_status() == 0


def test_self_test_argument_checks():
    w, cache, _, _ = _small_cache()
    for bad in (0, 1_000_001):
        with pytest.raises(KvsError) as e:
            cache.selftest_wait_timeout(bad)
        assert e.value.status == kb.KVS_ERR_INVALID_ARG
    assert cache.device_status() == 0
    ctx = kb.kvs_create(1, 1, 1, 64, 1, 8, kb.KVS_BF16, 0.0, 0)
    with pytest.raises(KvsError) as e:        # no memory bound yet
        kb.kvs_selftest_wait_timeout(ctx, 100)
    assert e.value.status == kb.KVS_ERR_STATE
    with pytest.raises(KvsError) as e:
        kb.kvs_clear_device_status(ctx)
    assert e.value.status == kb.KVS_ERR_STATE
    kb.kvs_destroy(ctx)


def test_bounds_self_test_is_refused_by_the_normal_build():
    if "bounds" in os.path.basename(kb.LIB_PATH):
        pytest.skip("the suite is running against the bounds-checking build (KVS_LIBRARY)")
    w, cache, _, _ = _small_cache()
    with pytest.raises(KvsError) as e:
        kb.kvs_selftest_bounds(cache.ctx)
    assert e.value.status == kb.KVS_ERR_STATE and cache.device_status() == 0


@pytest.mark.parametrize("Hq,Hkv,B,dtype,context", [(8, 8, 4, "bf16", 3000),      # scalar kernel, units < blocks: combine follows
                                                    (8, 8, 40, "bf16", 700),      # scalar kernel finishes the units itself
                                                    (16, 4, 2, "bf16", 9000),     # tensor-core kernel, combine follows
                                                    (16, 4, 64, "bf16", 500),     # tensor-core kernel finishes the units itself
                                                    (4, 4, 3, "f32", 2000)])
def test_a_withheld_copy_makes_the_attention_kernel_give_up_and_the_context_recovers(Hq, Hkv, B, dtype, context):
    """The give-up path of the real split-K kernels: one block's producer arms a tile's barrier and withholds
    the copies.  The consumers' wait runs out (2 ms), they hand the give-up to the producer, which waits for
    the copies it did issue; blocks that depend on the stalled one give up as well; the launch ends, the
    status word says TIMEOUT, and after kvs_clear_device_status the next call matches the oracle."""
    from paper_2410_18517_b200 import KVS_OPT_WAIT_LIMIT_US

    w = si.Workload(f"stall_{Hq}_{Hkv}_{B}_{dtype}", L=2, Hq=Hq, Hkv=Hkv, D=128, B=B, context=context, dtype=dtype,
                    n_shared=1, map_seed=0, steps=1, fixed_map=(0, 0))
    cache = SharedKVCache(w.L, w.Hq, w.Hkv, w.D, w.B, w.context + 4, w.dtype, share_map=w.share_map())
    k, v = si.context_kv(w, 0)
    cache.append(0, k.cuda(), v.cuda())
    q = si.step_qkv(w, 0, 1)[0]
    good = cache.decode_attention(1, q.cuda()).clone()
    cache.set_option(KVS_OPT_WAIT_LIMIT_US, 2000)
    out = torch.zeros_like(good)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    kb.kvs_selftest_stalled_copy(cache.ctx, 1, q.cuda(), out, w.B, torch.cuda.current_stream().cuda_stream)
    t1.record()
    torch.cuda.synchronize()
    assert cache.device_status() == kb.KVS_ERR_TIMEOUT
    assert 1.5 <= t0.elapsed_time(t1) <= 50.0          # it gave up after about the limit, not after seconds
    cache.clear_device_status()
    assert cache.device_status() == 0
    cache.set_option(KVS_OPT_WAIT_LIMIT_US, 2000000)
    again = cache.decode_attention(1, q.cuda())
    assert torch.equal(again, good)                      # the context works as before
    K, V = k.double().numpy(), v.double().numpy()
    rng = np.random.default_rng(0)
    for _ in range(6):
        b, hq = int(rng.integers(w.B)), int(rng.integers(w.Hq))
        ref = oracle.attend_unit(q[b, hq].double().numpy(), K[b, :, hq // w.G], V[b, :, hq // w.G])
        assert_close(again[b, hq].cpu().numpy(), ref, f"after the stalled launch, unit {(b, hq)}")
    assert cache.device_status() == 0
