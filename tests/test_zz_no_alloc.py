"""kvs_decode_attention_static: attention for callers that cannot allocate scratch memory.

Some users of this library run where device allocation is off the table: inside an engine
that has already claimed all free GPU memory for its own pools, or in a plug-in that is
handed tensors but no allocator.  For them the library carries a fixed 2 MiB scratch array
in its own image.  This test calls that entry point through the C ABI, twice in a row
(the array keeps the first call's leftovers, so the second call proves nothing stale is
used), and compares with the regular entry point, which takes its scratch from the bound
workspace.  Collected last on purpose: a failure here cannot hide another test's result.
"""
import pytest
import torch

import synth_inputs as si
from paper_2410_18517_b200 import SharedKVCache
from paper_2410_18517_b200 import binding as kb
from paper_2410_18517_b200 import build as kbuild

from helpers import MAX_ABS, REL_L2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


def _loaded_cache(w, extra=4):
    cache = SharedKVCache(w.L, w.Hq, w.Hkv, w.D, w.B, w.context + extra, w.dtype, share_map=w.share_map())
    for l in range(w.L):
        if w.share_map()[l] == l:
            k, v = si.context_kv(w, l, device="cuda")
            cache.append(l, k, v)
    return cache


@pytest.mark.parametrize("Hq,Hkv,dtype", [(8, 8, "bf16"), (8, 2, "bf16"), (4, 4, "f32")])
def test_static_scratch_matches_workspace_scratch_twice_in_a_row(Hq, Hkv, dtype):
    w = si.Workload(f"noalloc_{Hq}_{Hkv}_{dtype}", L=3, Hq=Hq, Hkv=Hkv, D=128, B=4, context=2500, dtype=dtype,
                    n_shared=1, map_seed=0, steps=1, fixed_map=(0, 1, 0))
    cache = _loaded_cache(w)
    stream = torch.cuda.current_stream().cuda_stream
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for call in range(2):
        # a different layer (and so a different slot, query and set of partial results) each call
        layer = (2, 1)[call]
        q = si.step_qkv(w, call, layer, device="cuda")[0]
        ref = cache.decode_attention(layer, q)
        out = torch.full_like(ref, float("nan"))
        kb.kvs_decode_attention_static(cache.ctx, layer, q, out, w.B, stream, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        err = (out - ref).abs().max().item()
        rel = ((out - ref).norm() / ref.norm()).item()
        assert err <= MAX_ABS and rel <= REL_L2, (call, err, rel)
        assert torch.equal(out, ref)          # same kernels, same split: the bits agree too
    # without a status pointer the call still works
    out2 = torch.empty_like(ref)
    kb.kvs_decode_attention_static(cache.ctx, layer, q, out2, w.B, stream, None)
    torch.cuda.synchronize()
    assert torch.equal(out2, ref)


def test_static_scratch_rejects_calls_beyond_its_size_and_bad_arguments():
    # 64 sequences x 64 kv-heads: 4096 units need more than 2 MiB of partial results
    big = SharedKVCache(1, 64, 64, 128, 64, 128, "bf16")
    k = torch.zeros(64, 8, 64, 128, dtype=torch.bfloat16, device="cuda")
    big.append(0, k, k)
    q = torch.zeros(64, 64, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.full((64, 64, 128), 7.0, dtype=torch.float32, device="cuda")
    launches = big.stats()["attention_launches"]
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_decode_attention_static(big.ctx, 0, q, out, 64, 0, None)
    assert e.value.status == kb.KVS_ERR_SCRATCH_LIMIT
    assert "scratch" in kb.kvs_status_string(kb.KVS_ERR_SCRATCH_LIMIT)
    torch.cuda.synchronize()
    assert big.stats()["attention_launches"] == launches and bool((out == 7.0).all())
    # the regular entry point handles the same call
    assert torch.isfinite(big.decode_attention(0, q)).all()
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_decode_attention_static(big.ctx, 3, q, out, 64, 0, None)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_decode_attention_static(big.ctx, 0, None, out, 64, 0, None)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG
