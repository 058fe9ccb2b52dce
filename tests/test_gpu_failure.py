"""Failure detection on the device: the give-up path of the bounded waits.

Every wait inside the pipelined kernels is bounded.  Nothing in the normal tests ever makes one
run out, so this file makes one run out on purpose, in the harmless way: a one-warp self-test kernel
waits, with a limit of about a millisecond, on a barrier that nothing arrives at (no copy is in
flight, nothing traps), through the very function the attention kernels wait with.  The wait gives
up, the status word reads KVS_ERR_TIMEOUT, the kernel returns, and the context goes on working.
"""
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
    w, cache, _, _ = _small_cache()
    with pytest.raises(KvsError) as e:
        kb.kvs_selftest_bounds(cache.ctx)
    assert e.value.status == kb.KVS_ERR_STATE and cache.device_status() == 0
