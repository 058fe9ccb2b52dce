"""Eviction and ragged slots on the GPU against the oracle: an outside intra-layer method decides
which rows of a computing layer's cache survive; sharing layers read the sparsified slot as is."""
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


def _random_keep(rng, B, Hkv, lens, lo_frac):
    stride = int(lens.max())
    n_keep = np.zeros((B, Hkv), dtype=np.int32)
    keep = np.zeros((B, Hkv, stride), dtype=np.int32)
    for b in range(B):
        for h in range(Hkv):
            n = int(lens[b, h])
            n_keep[b, h] = rng.integers(max(1, int(n * lo_frac)), n + 1)
            keep[b, h, : n_keep[b, h]] = np.sort(rng.choice(n, size=n_keep[b, h], replace=False))
    return keep, n_keep


def _check_state(cache, orc, w, sm, computing_only=False):
    """Lengths and cached bits, unit by unit.  Right after an eviction only the computing layers are
    compared: the oracle's sharing layer still holds its literal copy from its last turn and catches
    up at its next one, while the library's sharing layer reads the shared slot at once."""
    for l in range(w.L):
        if computing_only and sm[l] != l:
            continue
        K, V = orc.cache(l)
        s = cache.slot_of_layer(l)
        assert cache.seq_len(l) == orc.length(l)
        for b in range(w.B):
            for h in range(w.Hkv):
                n = orc.unit_len(l, b, h)
                assert cache.unit_len(l, b, h) == n
                gk = cache.plane(s, 0)[b, h, :n].double().cpu().numpy()
                gv = cache.plane(s, 1)[b, h, :n].double().cpu().numpy()
                assert np.array_equal(gk, K[b, h, :n]) and np.array_equal(gv, V[b, h, :n]), (l, b, h)


@pytest.mark.parametrize("dtype,D,Hq,Hkv", [("bf16", 128, 4, 2), ("bf16", 128, 8, 2), ("bf16", 64, 8, 1), ("f32", 64, 2, 2)])
@pytest.mark.parametrize("context,lo_frac", [(300, 0.5), (700, 0.05)])
def test_evict_then_decode_with_sharing(dtype, D, Hq, Hkv, context, lo_frac):
    sm = [0, 1, 2, 1]
    w = si.Workload(f"rag_{dtype}_{D}_{Hq}_{Hkv}_{context}", L=4, Hq=Hq, Hkv=Hkv, D=D, B=2, context=context, dtype=dtype,
                    n_shared=1, map_seed=0, steps=6, fixed_map=tuple(sm))
    rng = np.random.default_rng(context + Hq)
    cache = SharedKVCache(w.L, Hq, Hkv, D, w.B, context + 8, dtype, share_map=sm)
    orc = oracle.Oracle(w.L, Hq, Hkv, D, w.B, sm)
    for l in range(w.L):
        k, v = si.context_kv(w, l)
        orc.layer_forward(l, None, k.double().numpy(), v.double().numpy())
        cache.append(l, k.cuda(), v.cuda())

    def step(t):
        for l in range(w.L):
            q, k, v = si.step_qkv(w, t, l)
            ref = orc.layer_forward(l, q.double().numpy(), k.double().numpy(), v.double().numpy())
            cache.append(l, k.cuda(), v.cuda())
            assert_close(cache.decode_attention(l, q.cuda()).cpu().numpy(), ref, f"step {t} layer {l}")

    step(0)
    for round_ in range(2):                      # evict layer 1 twice (the second time it is already ragged)
        lens = np.array([[orc.unit_len(1, b, h) for h in range(Hkv)] for b in range(w.B)])
        keep, n_keep = _random_keep(rng, w.B, Hkv, lens, lo_frac)
        orc.evict(1, keep, n_keep)
        cache.evict(1, torch.from_numpy(keep).cuda(), n_keep)
        _check_state(cache, orc, w, sm, computing_only=True)
        step(1 + 2 * round_)
        step(2 + 2 * round_)
        _check_state(cache, orc, w, sm)
    assert cache.device_status() == 0
    assert cache.stats()["evict_launches"] == 2
    # a uniform layer next to the ragged one is untouched
    assert cache.unit_len(0, 1, 0) == context + 5 == cache.seq_len(0)


@pytest.mark.parametrize("Hq,Hkv,kernel", [(8, 8, 1), (32, 8, 2), (16, 4, 1)])
def test_ragged_slots_at_sizes_where_a_block_spans_several_units(Hq, Hkv, kernel):
    """64 or 32 units of up to 3000 rows cut to random lengths between 5 % and 100 %: every thread
    block's share of the tile line crosses units, many of its tiles lie past a unit's end, and units
    are shared by several blocks.  Inputs are made on the GPU; sampled (sequence, q-head) pairs are
    checked against the oracle run as a one-head problem on the kept rows sliced from those inputs,
    on the computing layer and on the layer that shares its slot, before and after two appends."""
    D, B, n = 128, 8, 3000
    sm = [0, 0]
    cache = SharedKVCache(2, Hq, Hkv, D, B, n + 4, "bf16", share_map=sm)
    cache.set_option(kb.KVS_OPT_KERNEL, kernel)
    k = si.normal((9, "rag_big_k", Hq, Hkv), (B, n, Hkv, D), torch.bfloat16, device="cuda")
    v = si.normal((9, "rag_big_v", Hq, Hkv), (B, n, Hkv, D), torch.bfloat16, device="cuda")
    cache.append(0, k, v)
    rng = np.random.default_rng(Hq * 100 + Hkv)
    keep, n_keep = _random_keep(rng, B, Hkv, np.full((B, Hkv), n), 0.05)
    cache.evict(0, torch.from_numpy(keep).cuda(), n_keep)
    G = Hq // Hkv
    pairs = sorted({(0, 0), (B - 1, Hq - 1)} | {(int(rng.integers(B)), int(rng.integers(Hq))) for _ in range(10)})
    new_k, new_v = [], []
    for step in range(3):
        q = si.normal((9, "rag_big_q", Hq, step), (B, Hq, D), torch.bfloat16, device="cuda")
        outs = [cache.decode_attention(l, q) for l in range(2)]
        assert torch.equal(outs[0].view(torch.int32), outs[1].view(torch.int32))     # the sharing layer reads the same slot
        assert cache.last_launch()["kernel"] == kernel
        for b, hq in pairs:
            hk = hq // G
            rows = torch.from_numpy(keep[b, hk, : n_keep[b, hk]].astype(np.int64)).cuda()
            kk = torch.cat([k[b, rows, hk]] + [t[b, :, hk] for t in new_k]).double().cpu().numpy()[None, :, None, :]
            vv = torch.cat([v[b, rows, hk]] + [t[b, :, hk] for t in new_v]).double().cpu().numpy()[None, :, None, :]
            one = oracle.Oracle(1, 1, 1, D, 1, [0])
            ref = one.layer_forward(0, q[b : b + 1, hq : hq + 1].double().cpu().numpy(), kk, vv)
            assert_close(outs[0][b : b + 1, hq : hq + 1].cpu().numpy(), ref, f"step {step} sequence {b} head {hq}")
            assert cache.unit_len(0, b, hk) == n_keep[b, hk] + step
        k1 = si.normal((9, "rag_big_k1", Hq, step), (B, 1, Hkv, D), torch.bfloat16, device="cuda")
        v1 = si.normal((9, "rag_big_v1", Hq, step), (B, 1, Hkv, D), torch.bfloat16, device="cuda")
        cache.append(0, k1, v1)
        new_k.append(k1)
        new_v.append(v1)
    assert cache.device_status() == 0


def test_evict_argument_checks_and_bad_lists():
    sm = [0, 0]
    cache = SharedKVCache(2, 2, 2, 128, 1, 64, "bf16", share_map=sm)
    keep = torch.arange(8, dtype=torch.int32, device="cuda").repeat(1, 2, 1).contiguous()
    with pytest.raises(KvsError) as e:                  # empty slot
        cache.evict(0, keep, [[4, 4]])
    assert e.value.status == kb.KVS_ERR_STATE
    k = torch.randn(1, 8, 2, 128, device="cuda").bfloat16()
    cache.append(0, k, k)
    with pytest.raises(KvsError) as e:                  # a sharing layer owns no cache
        cache.evict(1, keep, [[4, 4]])
    assert e.value.status == kb.KVS_ERR_INVALID_ARG
    for bad in ([[0, 4]], [[9, 4]]):                     # empty unit; more rows than cached
        with pytest.raises(KvsError) as e:
            cache.evict(0, keep, bad)
        assert e.value.status == kb.KVS_ERR_INVALID_ARG
    torch.cuda.synchronize()
    before = cache.pool.clone()
    # an out-of-range entry is only visible on the device: flagged there, that entry is skipped
    bad_keep = keep.clone()
    bad_keep[0, 0, 2] = 50
    cache.evict(0, bad_keep, [[4, 4]])
    assert cache.device_status() == kb.KVS_ERR_INVALID_ARG
    assert cache.unit_len(0, 0, 0) == 4 and cache.seq_len(1) == 4
    # rows 0,1,3 of unit (0,0) and 0..3 of unit (0,1) are what the lists said
    plane_before = before[: cache.plane(0, 0).numel() * 2].view(torch.bfloat16).view(1, 2, 128, 128)
    assert torch.equal(cache.plane(0, 0)[0, 1, :4], plane_before[0, 1, :4])
    assert torch.equal(cache.plane(0, 0)[0, 0, 3], plane_before[0, 0, 3])
    with pytest.raises(KvsError) as e:                  # no positions any more: no prefill
        cache.prefill_attention(0, torch.zeros(1, 2, 2, 128, dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == kb.KVS_ERR_STATE
    cache.reset()
    assert cache.unit_len(0, 0, 0) == 0
