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
@pytest.mark.parametrize("use_step", [False, True])
def test_graph_replay_is_the_next_step_every_time(Hq, Hkv, dtype, context, evict, use_step):
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
            if use_step:                         # kvs_decode_step: the append rides in the attention kernel
                own = sm[l] == l
                cache.decode_step(l, qb[l], kbuf[l] if own else None, vbuf[l] if own else None, ob[l])
                continue
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


@pytest.mark.parametrize("Hq,Hkv,evict,use_step", [(4, 4, False, False), (8, 2, False, False), (4, 2, True, False),
                                                    (4, 4, False, True), (8, 2, False, True)])
def test_replays_past_the_capacity_stop_appending_and_report(Hq, Hkv, evict, use_step):
    """Capacity 128 rows (one whole row stride), 126 cached, the recorded step makes 127: the replays
    after the first would need rows 128, 129, ...  The kernels' own checks append nothing there, attend
    over the rows that exist, set the status word, and the commit refuses; no row outside a unit is
    touched (the neighbouring units and the rest of the pool keep their bits)."""
    L, D, B, cap = 2, 128, 2, 128
    sm = [0, 0]
    w = si.Workload(f"replay_over_{Hq}_{Hkv}", L=L, Hq=Hq, Hkv=Hkv, D=D, B=B, context=cap - 2, dtype="bf16", n_shared=1,
                    map_seed=0, steps=8, fixed_map=tuple(sm))
    cache = SharedKVCache(L, Hq, Hkv, D, B, cap, "bf16", share_map=sm)
    cache.set_option(KVS_OPT_REPLAY, 1)
    k, v = si.context_kv(w, 0)
    cache.append(0, k.cuda(), v.cuda())
    if evict:                                     # a ragged slot: the longest unit keeps every row
        n_keep = np.full((B, Hkv), cap - 2, dtype=np.int32)
        n_keep[0, 0] = 40
        keep = np.tile(np.arange(cap - 2, dtype=np.int32), (B, Hkv, 1))
        cache.evict(0, torch.from_numpy(keep).cuda(), n_keep)
    q, kk, vv = (t.cuda() for t in si.step_qkv(w, 0, 0))
    out = torch.empty(B, Hq, D, dtype=torch.float32, device="cuda")

    def one_step():
        if use_step:
            cache.decode_step(0, q, kk, vv, out)
        else:
            cache.append(0, kk, vv)
            cache.decode_attention(0, q, out)
        cache.decode_attention(1, q, out)
        cache.replay_advance()

    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            one_step()
    before = cache.pool.clone()
    for _ in range(5):                            # rows 126, 127 fit; 128.. do not
        graph.replay()
    torch.cuda.synchronize()
    assert cache.device_status() == kb.KVS_ERR_CAPACITY
    with pytest.raises(KvsError) as e:
        cache.replay_commit(5)
    assert e.value.status == kb.KVS_ERR_CAPACITY
    assert torch.isfinite(out).all()
    # only the rows the replays could legally append may differ from the pool before the replays:
    # rows 126 and 127 of a full unit, rows 40..44 of the unit that was cut to 40 rows
    changed = (cache.pool != before).view(1, 2, B, Hkv, cap, D * 2).any(dim=-1)
    expect = torch.zeros_like(changed)
    expect[..., cap - 2 :] = True
    if evict:
        expect[:, :, 0, 0, :] = False
        expect[:, :, 0, 0, 40:45] = True
    assert torch.equal(changed, expect)


@pytest.mark.parametrize("Hq,Hkv,B", [(8, 8, 8), (32, 8, 4), (8, 8, 24), (32, 8, 24)])
def test_graph_replay_at_a_size_that_fills_the_gpu(Hq, Hkv, B):
    """32 or 64 units of about 2000 rows: every SM has a thread block, blocks span units, and the tile
    line is recomputed on the device from the replay counter (the context ends three rows before a
    tile boundary, so the replays cross it).  With batch 24 there are 192 units, more than thread blocks:
    the split-K kernel finishes the units itself (no combine launch; the hand-over flags must be back
    to zero after every replay).  Sampled (sequence, q-head) pairs of the computing layer
    and of the layer sharing its slot are checked against the oracle after every replay."""
    L, D, context, replays = 2, 128, 2045, 5
    sm = [0, 0]
    cache = SharedKVCache(L, Hq, Hkv, D, B, context + replays + 2, "bf16", share_map=sm)
    cache.set_option(KVS_OPT_REPLAY, 1)
    k = si.normal((13, "rp_big_k", Hq), (B, context, Hkv, D), torch.bfloat16, device="cuda")
    v = si.normal((13, "rp_big_v", Hq), (B, context, Hkv, D), torch.bfloat16, device="cuda")
    cache.append(0, k, v)
    qb = torch.empty(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    kbuf = torch.empty(B, 1, Hkv, D, dtype=torch.bfloat16, device="cuda")
    vbuf = torch.empty_like(kbuf)
    ob = [torch.empty(B, Hq, D, dtype=torch.float32, device="cuda") for _ in range(L)]
    rng = np.random.default_rng(Hq)
    G = Hq // Hkv
    pairs = sorted({(0, 0), (B - 1, Hq - 1)} | {(int(rng.integers(B)), int(rng.integers(Hq))) for _ in range(6)})
    ks, vs = [k], [v]

    def fill(t):
        qb.copy_(si.normal((13, "rp_big_q", Hq, t), (B, Hq, D), torch.bfloat16, device="cuda"))
        kbuf.copy_(si.normal((13, "rp_big_k1", Hq, t), (B, 1, Hkv, D), torch.bfloat16, device="cuda"))
        vbuf.copy_(si.normal((13, "rp_big_v1", Hq, t), (B, 1, Hkv, D), torch.bfloat16, device="cuda"))
        ks.append(kbuf.clone())
        vs.append(vbuf.clone())

    def one_step():
        cache.append(0, kbuf, vbuf)
        cache.decode_attention(0, qb, ob[0])
        cache.decode_attention(1, qb, ob[1])
        cache.replay_advance()

    def check(what):
        torch.cuda.synchronize()
        assert torch.equal(ob[0].view(torch.int32), ob[1].view(torch.int32))
        kall, vall = torch.cat(ks, dim=1), torch.cat(vs, dim=1)
        for b, hq in pairs:
            hk = hq // G
            one = oracle.Oracle(1, 1, 1, D, 1, [0])
            ref = one.layer_forward(0, qb[b : b + 1, hq : hq + 1].double().cpu().numpy(),
                                    kall[b : b + 1, :, hk : hk + 1].double().cpu().numpy(),
                                    vall[b : b + 1, :, hk : hk + 1].double().cpu().numpy())
            assert_close(ob[0][b : b + 1, hq : hq + 1].cpu().numpy(), ref, f"{what} sequence {b} head {hq}")

    fill(0)
    one_step()                                   # eager
    check("eager step")
    fill(1)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            one_step()
    for r in range(replays):
        if r > 0:
            fill(1 + r)
        graph.replay()
        check(f"replay {r}")
    cache.replay_commit(replays)
    torch.cuda.synchronize()
    assert cache.device_status() == 0 and cache.seq_len(1) == context + 1 + replays
    assert (cache.stats()["combine_launches"] == 0) == (B * Hkv >= 148)
    kall = torch.cat(ks, dim=1)
    assert torch.equal(cache.plane(0, 0)[:B, :, : context + 1 + replays], kall.permute(0, 2, 1, 3))
