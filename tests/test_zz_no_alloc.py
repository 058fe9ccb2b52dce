"""kvs_decode_attention_static: attention for callers that cannot allocate scratch memory.

Some users of this library run where device allocation is off the table: inside an engine
that has already claimed all free GPU memory for its own pools, or in a plug-in that is
handed tensors but no allocator.  For them the library carries a fixed 2 MiB scratch array
in its own image.  This test calls that entry point through the C ABI, twice in a row
(the array keeps the first call's leftovers, so the second call proves nothing stale is
used), and compares with the regular entry point, which takes its scratch from the bound
workspace, and with the fp64 oracle.  Collected last on purpose: a failure here cannot hide
another test's result.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_2410_18517_b200 import SharedKVCache
from paper_2410_18517_b200 import binding as kb
from paper_2410_18517_b200 import build as kbuild

from helpers import MAX_ABS, REL_L2, assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


def _loaded_cache(w, extra=4):
    """The cache plus the context rows of every computing layer (kept for the oracle)."""
    cache = SharedKVCache(w.L, w.Hq, w.Hkv, w.D, w.B, w.context + extra, w.dtype, share_map=w.share_map())
    rows = {}
    for l in range(w.L):
        if w.share_map()[l] == l:
            k, v = si.context_kv(w, l, device="cuda")
            cache.append(l, k, v)
            rows[l] = (k.double().cpu().numpy(), v.double().cpu().numpy())
    return cache, rows


def _check_units_against_oracle(w, layer, q, K, V, out, what, n_units=6):
    """A few (sequence, q-head) units of `out` against the definition in fp64."""
    rng = np.random.default_rng(layer)
    qd, od = q.double().cpu().numpy(), out.cpu().numpy()
    for _ in range(n_units):
        b, hq = int(rng.integers(0, w.B)), int(rng.integers(0, w.Hq))
        ref = oracle.attend_unit(qd[b, hq], K[b, :, hq // w.G], V[b, :, hq // w.G])
        assert_close(od[b, hq], ref, f"{what}, unit {(b, hq)}")


@pytest.mark.parametrize("Hq,Hkv,dtype", [(8, 8, "bf16"), (8, 2, "bf16"), (4, 4, "f32")])
def test_static_scratch_matches_workspace_scratch_twice_in_a_row(Hq, Hkv, dtype):
    w = si.Workload(f"noalloc_{Hq}_{Hkv}_{dtype}", L=3, Hq=Hq, Hkv=Hkv, D=128, B=4, context=2500, dtype=dtype,
                    n_shared=1, map_seed=0, steps=1, fixed_map=(0, 1, 0))
    cache, rows = _loaded_cache(w)
    stream = torch.cuda.current_stream().cuda_stream
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
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
        # and against the definition: layer 2 reads layer 0's cache, layer 1 its own
        K, V = rows[int(w.share_map()[layer])]
        _check_units_against_oracle(w, layer, q, K, V, out, f"static call {call}")
    # without a status pointer the call still works
    out2 = torch.empty_like(ref)
    kb.kvs_decode_attention_static(cache.ctx, layer, q, out2, w.B, stream, None)
    torch.cuda.synchronize()
    assert torch.equal(out2, ref)
    # The device as a whole holds no more memory than before the calls: torch's own tensors come
    # from its cached pool, and the library reserved nothing (driver-level free memory unchanged).
    assert torch.cuda.mem_get_info()[0] >= free_before


def test_static_calls_of_different_sizes_share_the_array():
    """A call with few units, whose partial results fill the front of the array, then one with hundreds of
    units that hands pieces over through per-unit flags, then the small one again: the flags of the large
    call lie where no call keeps partial results, so nothing the small call left can be read as a flag."""
    small = si.Workload("noalloc_small", L=1, Hq=8, Hkv=2, D=128, B=4, context=3000, dtype="bf16",
                        n_shared=0, map_seed=0, steps=1, fixed_map=(0,))
    large = si.Workload("noalloc_large", L=1, Hq=32, Hkv=8, D=128, B=32, context=700, dtype="bf16",
                        n_shared=0, map_seed=0, steps=1, fixed_map=(0,))
    made = [(w,) + _loaded_cache(w) for w in (small, large)]
    stream = torch.cuda.current_stream().cuda_stream
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for rep, (w, cache, rows) in enumerate([made[0], made[1], made[0], made[1]]):
        q = si.step_qkv(w, rep, 0, device="cuda")[0]
        ref = cache.decode_attention(0, q)
        out = torch.full_like(ref, float("nan"))
        kb.kvs_decode_attention_static(cache.ctx, 0, q, out, w.B, stream, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(out, ref), rep
        K, V = rows[0]
        _check_units_against_oracle(w, 0, q, K, V, out, f"call {rep} ({w.name})")
    assert made[1][1].stats()["combine_launches"] == 0      # the large calls were finished inside the split-K kernel


def test_static_call_on_a_second_stream_beside_the_contexts_chain():
    """A decode step on stream A (the append rides in the attention kernel), the static call on
    stream B after an event, then the next decode step on A without waiting for B: the static call
    must not disturb what A's next kernel believes it may fetch early.  All three against the oracle."""
    w = si.Workload("noalloc_two_streams", L=2, Hq=8, Hkv=2, D=128, B=4, context=1900, dtype="bf16",
                    n_shared=1, map_seed=0, steps=2, fixed_map=(0, 0))
    cache, rows = _loaded_cache(w, extra=8)
    K, V = rows[0]
    A, B = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = []
    for rep in range(4):
        q0, k0, v0 = si.step_qkv(w, 2 * rep, 0, device="cuda")
        q1 = si.step_qkv(w, 2 * rep, 1, device="cuda")[0]
        q2, k2, v2 = si.step_qkv(w, 2 * rep + 1, 0, device="cuda")
        torch.cuda.synchronize()
        with torch.cuda.stream(A):
            o0 = cache.decode_step(0, q0, k0, v0)
            ev = torch.cuda.Event()
            ev.record(A)
        B.wait_event(ev)
        o1 = torch.empty_like(o0)
        kb.kvs_decode_attention_static(cache.ctx, 1, q1, o1, w.B, B.cuda_stream, None)
        with torch.cuda.stream(A):
            o2 = cache.decode_step(0, q2, k2, v2)
        torch.cuda.synchronize()
        K = np.concatenate([K, k0.double().cpu().numpy()], axis=1)
        Vn = np.concatenate([V, v0.double().cpu().numpy()], axis=1)
        _check_units_against_oracle(w, 0, q0, K, Vn, o0, f"rep {rep}: step on A")
        _check_units_against_oracle(w, 1, q1, K, Vn, o1, f"rep {rep}: static call on B")
        K = np.concatenate([K, k2.double().cpu().numpy()], axis=1)
        V = np.concatenate([Vn, v2.double().cpu().numpy()], axis=1)
        _check_units_against_oracle(w, 0, q2, K, V, o2, f"rep {rep}: next step on A")
        outs.append((o0, o1, o2))
    assert cache.device_status() == 0


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
    # a status pointer that is not 4-byte aligned is refused before anything is launched
    small = SharedKVCache(1, 4, 4, 128, 2, 64, "bf16")
    ks = torch.zeros(2, 8, 4, 128, dtype=torch.bfloat16, device="cuda")
    small.append(0, ks, ks)
    qs = torch.zeros(2, 4, 128, dtype=torch.bfloat16, device="cuda")
    os_ = torch.full((2, 4, 128), 7.0, dtype=torch.float32, device="cuda")
    word = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_decode_attention_static(small.ctx, 0, qs, os_, 2, 0, word.data_ptr() + 2)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert bool((os_ == 7.0).all())
