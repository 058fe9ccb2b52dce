"""The one-kernel decode step (thread-block cluster per unit, append and merge inside the kernel)
against the fp64 oracle, and against the three-kernel path it replaces."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from paper_2410_18517_b200 import KVS_OPT_EARLY_START, KVS_OPT_KERNEL, KvsError, SharedKVCache
from paper_2410_18517_b200 import build as kbuild

from helpers import make_cache, run_small

pytestmark = pytest.mark.gpu

CLUSTER = [(KVS_OPT_KERNEL, 3)]


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


@pytest.mark.parametrize("dtype,D,Hq,Hkv", [("bf16", 128, 4, 4), ("bf16", 128, 8, 2), ("bf16", 128, 8, 1), ("bf16", 128, 4, 2),
                                             ("bf16", 64, 4, 4), ("bf16", 64, 8, 2), ("f32", 64, 2, 2), ("f32", 128, 4, 1)])
@pytest.mark.parametrize("context", [0, 1, 63, 64, 65, 200, 1031, 4100])
def test_decode_step_in_one_kernel(dtype, D, Hq, Hkv, context):
    """Every output and every cached bit over five steps that cross tile boundaries: the appended
    row is attended to from the caller's buffer and must also land in the slot, where the sharing
    layer and the later steps read it."""
    w = si.Workload(f"cl_{dtype}_{D}_{Hq}_{Hkv}_{context}", L=3, Hq=Hq, Hkv=Hkv, D=D, B=2, context=context, dtype=dtype,
                    n_shared=1, map_seed=0, steps=5, fixed_map=(0, 1, 0))
    cache, _, _ = run_small(w, steps=5, options=CLUSTER, use_step=True)
    assert cache.last_launch()["kernel"] == 3
    st = cache.stats()
    assert st["fused_appends"] == 10 and st["combine_launches"] == 0
    assert st["append_skipped"] == 5 + (1 if context else 0)         # the sharing layer: every step, and the context load
    assert st["append_launches"] == (2 if context else 0)            # the context loads only


@pytest.mark.parametrize("Hq,Hkv,B,context", [(8, 2, 1, 9000), (4, 4, 3, 700), (8, 8, 1, 30000), (2, 1, 1, 70000)])
def test_clusters_of_every_size(Hq, Hkv, B, context):
    """Few units and long caches give clusters of 16 blocks with many tiles each; many units give
    small clusters."""
    w = si.Workload(f"cls_{Hq}_{Hkv}_{B}_{context}", L=2, Hq=Hq, Hkv=Hkv, D=128, B=B, context=context, dtype="bf16",
                    n_shared=1, map_seed=0, steps=2, fixed_map=(0, 0))
    cache, _, _ = run_small(w, steps=2, options=CLUSTER, use_step=True)
    ll = cache.last_launch()
    assert ll["kernel"] == 3 and ll["ctas"] % (B * Hkv) == 0 and 1 <= ll["ctas"] // (B * Hkv) <= 16


@pytest.mark.parametrize("early", [0, 1])
def test_attention_only_and_early_start(early):
    """kvs_append + kvs_decode_attention with the cluster kernel doing the attention, with and
    without early-start launches."""
    w = si.Workload(f"cl_att_{early}", L=4, Hq=8, Hkv=2, D=128, B=2, context=900, dtype="bf16", n_shared=2, map_seed=0,
                    steps=8, fixed_map=(0, 0, 2, 2))
    cache, _, _ = run_small(w, steps=8, options=CLUSTER + [(KVS_OPT_EARLY_START, early)])
    assert cache.last_launch()["kernel"] == 3 and cache.stats()["fused_appends"] == 0


def test_same_cache_bits_and_close_outputs_as_the_three_kernel_path():
    w = si.Workload("cl_vs_plain", L=3, Hq=8, Hkv=2, D=128, B=2, context=1500, dtype="bf16", n_shared=1, map_seed=0,
                    steps=4, fixed_map=(0, 1, 0))
    one, _, _ = run_small(w, steps=4, options=CLUSTER, use_step=True)
    three, _, _ = run_small(w, steps=4, options=[(KVS_OPT_KERNEL, 1)], use_step=True, check_cache=False)
    assert three.stats()["fused_appends"] == 0 and three.stats()["combine_launches"] == 12
    for s in range(2):
        for kv in range(2):
            assert torch.equal(one.plane(s, kv), three.plane(s, kv))
    q = si.step_qkv(w, 50, 2, device="cuda")[0]
    a, b = one.decode_attention(2, q), three.decode_attention(2, q)
    assert float((a - b).abs().max()) < 1e-5


def test_auto_choice_by_size_and_fallbacks():
    """Small launches take the cluster kernel by themselves; large ones, evicted slots and groups the
    cluster kernel does not have fall back to the other kernels, also through kvs_decode_step."""
    small = si.Workload("cl_auto_small", L=2, Hq=8, Hkv=2, D=128, B=2, context=500, dtype="bf16", n_shared=1, map_seed=0,
                        steps=2, fixed_map=(0, 0))
    cache, _, _ = run_small(small, steps=2, use_step=True)
    assert cache.last_launch()["kernel"] == 3
    big = si.Workload("cl_auto_big", L=1, Hq=8, Hkv=8, D=128, B=8, context=3000, dtype="bf16", n_shared=0, map_seed=0, steps=1)
    cache, _, _ = run_small(big, steps=1, use_step=True)       # 2*64*3000*256 B = 98 MB
    assert cache.last_launch()["kernel"] == 1 and cache.stats()["fused_appends"] == 0
    odd = si.Workload("cl_auto_odd", L=2, Hq=6, Hkv=2, D=128, B=2, context=300, dtype="bf16", n_shared=1, map_seed=0,
                      steps=2, fixed_map=(0, 0))
    cache, _, _ = run_small(odd, steps=2, use_step=True)
    assert cache.last_launch()["kernel"] == 2
    with pytest.raises(KvsError):
        cache.set_option(KVS_OPT_KERNEL, 3)                      # groups of 3 q-heads: no cluster kernel


def test_decode_step_argument_checks():
    w = si.Workload("cl_args", L=2, Hq=4, Hkv=2, D=64, B=2, context=8, dtype="bf16", n_shared=1, map_seed=0, steps=1,
                    fixed_map=(0, 0))
    cache = make_cache(w, 1)
    q, k, v = si.step_qkv(w, 0, 0, device="cuda")
    with pytest.raises(KvsError):
        cache.decode_step(1, q)                                  # sharing layer, but its source is still empty
    out = cache.decode_step(0, q, k, v)                          # first row of an empty slot
    assert cache.seq_len(0) == 1 and cache.seq_len(1) == 1
    ref = v.float()[:, 0].repeat_interleave(2, dim=1)            # one cached row: the output is that value row
    assert torch.allclose(out, ref, atol=1e-6)
    with pytest.raises(KvsError):
        cache.decode_step(0, q, None, None)                      # a computing layer needs k and v
    with pytest.raises(KvsError):
        cache.decode_step(5, q, k, v)
    for _ in range(8):
        cache.decode_step(0, q, k, v)
    with pytest.raises(KvsError):
        cache.decode_step(0, q, k, v)                            # capacity (8 + 1 rows)
    assert cache.seq_len(0) == 9 and cache.device_status() == 0
