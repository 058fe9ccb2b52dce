"""kvs_decode_step: the append of a decode step riding in the split-K attention kernel, against the
fp64 oracle and, bit for bit, against kvs_append + kvs_decode_attention."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from paper_2410_18517_b200 import KVS_OPT_EARLY_START, KVS_OPT_KERNEL, KvsError, SharedKVCache
from paper_2410_18517_b200 import build as kbuild

from helpers import make_cache, run_small

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


@pytest.mark.parametrize("dtype,D,Hq,Hkv,kernel", [("bf16", 128, 4, 4, 1), ("bf16", 128, 8, 2, 2), ("bf16", 128, 8, 2, 1),
                                                    ("bf16", 128, 8, 1, 2), ("bf16", 128, 6, 2, 2), ("bf16", 64, 4, 4, 1),
                                                    ("bf16", 64, 8, 2, 2), ("f32", 64, 2, 2, 1), ("f32", 128, 4, 1, 1)])
@pytest.mark.parametrize("context", [0, 1, 63, 64, 127, 128, 200, 1031])
def test_decode_step_every_output_and_every_cached_bit(dtype, D, Hq, Hkv, kernel, context):
    """Five steps that cross tile boundaries on both split-K kernels: the new row must be attended to
    in the step that appends it and must be in the slot for the sharing layer and the later steps."""
    w = si.Workload(f"st_{dtype}_{D}_{Hq}_{Hkv}_{context}", L=3, Hq=Hq, Hkv=Hkv, D=D, B=2, context=context, dtype=dtype,
                    n_shared=1, map_seed=0, steps=5, fixed_map=(0, 1, 0))
    cache, _, _ = run_small(w, steps=5, options=[(KVS_OPT_KERNEL, kernel)], use_step=True)
    assert cache.last_launch()["kernel"] == kernel
    st = cache.stats()
    # a call with no more thread blocks than units needs no combine launch (the short contexts here)
    assert st["fused_appends"] == 10 and st["combine_launches"] <= 15 and st["attention_launches"] == 15
    assert st["append_launches"] == (2 if context else 0)            # the context loads only


@pytest.mark.parametrize("Hq,Hkv,B,context", [(8, 8, 8, 300), (8, 2, 1, 9000), (32, 8, 16, 70), (4, 4, 3, 2500)])
@pytest.mark.parametrize("early", [0, 1])
def test_same_bits_as_append_then_attention(Hq, Hkv, B, context, early):
    """Many units per thread block, many thread blocks per unit, early-start launches on and off:
    outputs and the whole pool must equal those of the separate calls bit for bit over four steps."""
    w = si.Workload(f"st_eq_{Hq}_{Hkv}_{B}_{context}", L=3, Hq=Hq, Hkv=Hkv, D=128, B=B, context=context, dtype="bf16",
                    n_shared=1, map_seed=0, steps=4, fixed_map=(0, 1, 0))
    sm = w.share_map()
    one, two = make_cache(w, 4), make_cache(w, 4)
    for c in (one, two):
        c.set_option(KVS_OPT_EARLY_START, early)
    for l in range(w.L):
        if sm[l] == l:
            k, v = si.context_kv(w, l, device="cuda")
            one.append(l, k, v)
            two.append(l, k, v)
    for t in range(4):
        for l in range(w.L):
            q, k, v = si.step_qkv(w, t, l, device="cuda")
            own = sm[l] == l
            a = one.decode_step(l, q, k if own else None, v if own else None)
            if own:
                two.append(l, k, v)
            b = two.decode_attention(l, q)
            assert torch.equal(a.view(torch.int32), b.view(torch.int32)), (t, l)
    torch.cuda.synchronize()
    assert torch.equal(one.pool, two.pool)
    assert one.device_status() == 0 and one.stats()["fused_appends"] == 8 and two.stats()["fused_appends"] == 0


def test_full_size_layers_same_bits():
    """Four layers of the 7B shape (B=8, 32 heads, 4096 rows): every SM's block ends one or two units."""
    w = si.WORKLOADS["7b_mha_l4"]
    sm = w.share_map()
    one, two = make_cache(w, 4), make_cache(w, 4)
    for l in range(w.L):
        if sm[l] == l:
            k, v = si.context_kv(w, l, device="cuda")
            one.append(l, k, v)
            two.append(l, k, v)
    for t in range(3):
        for l in range(w.L):
            q, k, v = si.step_qkv(w, t, l, device="cuda")
            own = sm[l] == l
            a = one.decode_step(l, q, k if own else None, v if own else None)
            if own:
                two.append(l, k, v)
            assert torch.equal(a.view(torch.int32), two.decode_attention(l, q).view(torch.int32)), (t, l)
    torch.cuda.synchronize()
    assert torch.equal(one.pool, two.pool) and one.device_status() == 0


def test_decode_step_argument_checks_and_fallbacks():
    w = si.Workload("st_args", L=2, Hq=4, Hkv=2, D=64, B=2, context=8, dtype="bf16", n_shared=1, map_seed=0, steps=1,
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
    # an evicted (ragged) slot takes the separate append kernel
    n_keep = np.full((2, 2), 5, dtype=np.int32)
    keep = np.tile(np.arange(9, dtype=np.int32), (2, 2, 1))
    cache.evict(0, torch.from_numpy(keep).cuda(), n_keep)
    before = cache.stats()
    cache.decode_step(0, q, k, v)
    after = cache.stats()
    assert after["fused_appends"] == before["fused_appends"] and after["append_launches"] == before["append_launches"] + 1
    assert cache.unit_len(0, 0, 0) == 6
