"""A recorded decode step replayed as a CUDA graph: every replay must be the next decode step
(one row further, one row more attended), compared with the oracle stepping alongside."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_2410_18517_b200 import KVS_OPT_REPLAY, KvsError, SharedKVCache
from paper_2410_18517_b200 import binding as kb
from paper_2410_18517_b200 import build as kbuild

from helpers import assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


@pytest.mark.parametrize("Hq,Hkv,dtype,context,evict", [(4, 4, "bf16", 300, False), (8, 2, "bf16", 127, False),
                                                         (4, 2, "f32", 60, False), (8, 2, "bf16", 200, True)])
def test_graph_replay_is_the_next_step_every_time(Hq, Hkv, dtype, context, evict):
    sm = [0, 1, 2, 1]
    L, D, B, replays = 4, 128, 2, 6
    w = si.Workload(f"replay_{Hq}_{Hkv}_{dtype}", L=L, Hq=Hq, Hkv=Hkv, D=D, B=B, context=context, dtype=dtype,
                    n_shared=1, map_seed=0, steps=replays + 2, fixed_map=tuple(sm))
    cache = SharedKVCache(L, Hq, Hkv, D, B, context + replays + 2, dtype, share_map=sm)
    cache.set_option(KVS_OPT_REPLAY, 1)
    orc = oracle.Oracle(L, Hq, Hkv, D, B, sm)
    for l in range(L):
        k, v = si.context_kv(w, l)
        orc.layer_forward(l, None, k.double().numpy(), v.double().numpy())
        cache.append(l, k.cuda(), v.cuda())
    if evict:                                    # layer 1 (and its sharer, layer 3) become ragged first
        rng = np.random.default_rng(3)
        n_keep = rng.integers(context // 2, context + 1, size=(B, Hkv)).astype(np.int32)
        keep = np.zeros((B, Hkv, context), dtype=np.int32)
        for b in range(B):
            for h in range(Hkv):
                keep[b, h, : n_keep[b, h]] = np.sort(rng.choice(context, size=n_keep[b, h], replace=False))
        orc.evict(1, keep, n_keep)
        cache.evict(1, torch.from_numpy(keep).cuda(), n_keep)
    # device buffers the recorded launches read from and write to
    qb = [torch.empty(B, Hq, D, dtype=w.torch_dtype, device="cuda") for _ in range(L)]
    kbuf = [torch.empty(B, 1, Hkv, D, dtype=w.torch_dtype, device="cuda") for _ in range(L)]
    vbuf = [torch.empty(B, 1, Hkv, D, dtype=w.torch_dtype, device="cuda") for _ in range(L)]
    ob = [torch.empty(B, Hq, D, dtype=torch.float32, device="cuda") for _ in range(L)]

    def fill(t):
        refs = []
        for l in range(L):
            q, k, v = si.step_qkv(w, t, l)
            qb[l].copy_(q); kbuf[l].copy_(k); vbuf[l].copy_(v)
            refs.append(orc.layer_forward(l, q.double().numpy(), k.double().numpy(), v.double().numpy()))
        return refs

    def one_step():
        for l in range(L):
            if sm[l] == l:
                cache.append(l, kbuf[l], vbuf[l])
            else:
                cache.append(l, None, None, B, 1)
            cache.decode_attention(l, qb[l], ob[l])
        cache.replay_advance()

    def check(refs, what):
        torch.cuda.synchronize()
        for l in range(L):
            assert_close(ob[l].cpu().numpy(), refs[l], f"{what} layer {l}")

    refs = fill(0)
    one_step()                                   # eager: an ordinary step, the advance does nothing
    check(refs, "eager step")
    refs = fill(1)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            one_step()                           # recorded, not run
    assert cache.seq_len(0) == context + 2       # the bookkeeping counted the recorded step once
    for r in range(replays):
        if r > 0:
            refs = fill(1 + r)
        graph.replay()
        check(refs, f"replay {r}")
    cache.replay_commit(replays)
    torch.cuda.synchronize()
    assert cache.device_status() == 0
    for l in range(L):
        assert cache.seq_len(l) == orc.length(l)
        K, V = orc.cache(l)
        s = cache.slot_of_layer(l)
        for b in range(B):
            for h in range(Hkv):
                n = orc.unit_len(l, b, h)
                assert cache.unit_len(l, b, h) == n
                assert np.array_equal(cache.plane(s, 0)[b, h, :n].double().cpu().numpy(), K[b, h, :n])
                assert np.array_equal(cache.plane(s, 1)[b, h, :n].double().cpu().numpy(), V[b, h, :n])
    assert cache.seq_len(0) == context + 1 + replays
    refs = fill(1 + replays)                     # and eager steps continue from there
    one_step()
    check(refs, "eager step after commit")


def test_replay_calls_need_the_option():
    cache = SharedKVCache(1, 2, 2, 64, 1, 16, "bf16")
    with pytest.raises(KvsError) as e:
        cache.replay_advance()
    assert e.value.status == kb.KVS_ERR_STATE
    cache.set_option(KVS_OPT_REPLAY, 1)
    cache.replay_advance()                       # not capturing: nothing to do
    with pytest.raises(KvsError):
        cache.replay_commit(0)
    k = torch.zeros(1, 16, 2, 64, dtype=torch.bfloat16, device="cuda")
    cache.append(0, k, k)
    with pytest.raises(KvsError) as e:           # 16 rows cached, capacity 16: no room for 3 more
        cache.replay_commit(4)
    assert e.value.status == kb.KVS_ERR_CAPACITY
