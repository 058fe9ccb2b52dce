"""Parity of the tensor-core prefill kernel (through the C ABI) with the fp64 oracle: causal
attention of the newest n_q positions over the slot the layer's strategy entry points to."""
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


def _prefill_both(Hq, Hkv, B, chunks, share_map, seed=0, D=128, dtype="bf16"):
    """Feed the prompt in `chunks` (list of chunk lengths) to both sides, layer by layer."""
    L = len(share_map)
    total = sum(chunks)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    cache = SharedKVCache(L, Hq, Hkv, D, B, total, dtype, share_map=share_map)
    orc = oracle.Oracle(L, Hq, Hkv, D, B, share_map)
    worst = (0.0, 0.0)
    for c, T in enumerate(chunks):
        for l in range(L):
            w = si.Workload(f"pf_{seed}_{c}", L=L, Hq=Hq, Hkv=Hkv, D=D, B=B, context=T, dtype=dtype, n_shared=0,
                            map_seed=0, steps=1)
            k, v = si.context_kv(w, l, base_seed=seed)
            q = si.normal((seed, "pf_q", c, l), (B, T, Hq, D), tdt)
            ref = orc.layer_prefill(l, q.double().numpy(), k.double().numpy(), v.double().numpy())
            if share_map[l] == l:
                cache.append(l, k.cuda(), v.cuda())
            out = cache.prefill_attention(l, q.cuda())
            e = assert_close(out.cpu().numpy(), ref, f"chunk {c} layer {l}")
            worst = (max(worst[0], e[0]), max(worst[1], e[1]))
            assert cache.seq_len(l) == orc.length(l)
    assert cache.device_status() == 0
    return cache, orc, worst


def test_one_tile():
    _prefill_both(2, 2, 1, [128], [0])


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (4, 2), (8, 1)])
@pytest.mark.parametrize("chunks", [[1], [127], [129], [300], [512], [200, 333], [128, 1, 77]])
def test_prompt_lengths_chunks_and_sharing(Hq, Hkv, chunks):
    _prefill_both(Hq, Hkv, 2, chunks, [0, 0, 2, 0])


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (8, 2)])
@pytest.mark.parametrize("chunks", [[1], [64], [129], [300], [200, 333]])
def test_head_size_64(Hq, Hkv, chunks):
    _prefill_both(Hq, Hkv, 2, chunks, [0, 0, 2, 0], D=64)


@pytest.mark.parametrize("D,Hq,Hkv", [(64, 4, 4), (128, 4, 2), (128, 8, 1), (64, 2, 1)])
@pytest.mark.parametrize("chunks", [[1], [33], [128], [200, 77], [128, 1, 8]])
def test_fp32_storage(D, Hq, Hkv, chunks):
    """fp32 Q/K/V (the small configuration: 4 heads, head size 64, 128 context rows) go through the plain
    fp32 prefill kernel; same oracle, same strategy handling, and far inside the bf16 tolerance."""
    _, _, worst = _prefill_both(Hq, Hkv, 2, chunks, [0, 1, 2, 1], D=D, dtype="f32")
    assert worst[0] < 1e-4


@pytest.mark.parametrize("D,Hq,Hkv,B,chunks", [(128, 32, 8, 2, [2100]), (128, 16, 16, 3, [1500]), (64, 32, 8, 2, [2100]),
                                               (128, 32, 8, 2, [1000, 1100]),
                                               (128, 32, 32, 2, [4096])])   # the last one: the shape prefill_bench times
def test_many_items_per_block_sampled_heads(D, Hq, Hkv, B, chunks):
    """Sizes at which every persistent block works through several (query block, head) items one after the
    other (item ring, barrier phases and the output staging carried across items, K/V groups that do
    not all fit the scheduling group), with the prompt in one piece or in two.  The inputs are generated
    on the GPU; the oracle gets the rows of sampled (sequence, q-head) pairs sliced from those same
    tensors, each run as a one-head problem, and every query row of a sampled pair is compared."""
    sm = [0, 0]
    total = sum(chunks)
    cache = SharedKVCache(2, Hq, Hkv, D, B, total, "bf16", share_map=sm)
    G = Hq // Hkv
    rng = np.random.default_rng(11)
    pairs = sorted({(0, 0), (B - 1, Hq - 1)} | {(int(rng.integers(B)), int(rng.integers(Hq))) for _ in range(10)})
    ones = {p: oracle.Oracle(1, 1, 1, D, 1, [0]) for p in pairs}
    for c, T in enumerate(chunks):
        k = si.normal((5, "pf_big_k", D, Hq, total, c), (B, T, Hkv, D), torch.bfloat16, device="cuda")
        v = si.normal((5, "pf_big_v", D, Hq, total, c), (B, T, Hkv, D), torch.bfloat16, device="cuda")
        q = si.normal((5, "pf_big_q", D, Hq, total, c), (B, T, Hq, D), torch.bfloat16, device="cuda")
        cache.append(0, k, v)
        outs = [cache.prefill_attention(l % 2, q) for l in range(6)]  # own slot and the sharing layer in turn
        torch.cuda.synchronize()
        assert cache.device_status() == 0
        for o in outs[1:]:                                             # same slot, same queries: the same bits,
            assert torch.equal(o.view(torch.int32), outs[0].view(torch.int32))   # whichever block ran which item
        assert torch.isfinite(outs[0]).all()
        for b, hq in pairs:
            hk = hq // G
            ref = ones[(b, hq)].layer_prefill(0, q[b : b + 1, :, hq : hq + 1].double().cpu().numpy(),
                                              k[b : b + 1, :, hk : hk + 1].double().cpu().numpy(),
                                              v[b : b + 1, :, hk : hk + 1].double().cpu().numpy())
            assert_close(outs[0][b : b + 1, :, hq : hq + 1].cpu().numpy(), ref, f"chunk {c} sequence {b} head {hq}")


def test_prefill_then_decode_continues_from_the_same_cache():
    cache, orc, _ = _prefill_both(4, 2, 2, [260], [0, 1, 0])
    w = si.Workload("pf_dec", L=3, Hq=4, Hkv=2, D=128, B=2, context=0, dtype="bf16", n_shared=0, map_seed=0, steps=1)
    big = SharedKVCache(3, 4, 2, 128, 2, 300, "bf16", share_map=[0, 1, 0])
    # same prompt into a roomier cache, then two decode steps on both sides
    orc2 = oracle.Oracle(3, 4, 2, 128, 2, [0, 1, 0])
    wl = si.Workload("pf_0_0", L=3, Hq=4, Hkv=2, D=128, B=2, context=260, dtype="bf16", n_shared=0, map_seed=0, steps=1)
    for l in range(3):
        k, v = si.context_kv(wl, l)
        orc2.layer_forward(l, None, k.double().numpy(), v.double().numpy())
        if l != 2:
            big.append(l, k.cuda(), v.cuda())
    for t in range(2):
        for l in range(3):
            q, k, v = si.step_qkv(w, t, l)
            ref = orc2.layer_forward(l, q.double().numpy(), k.double().numpy(), v.double().numpy())
            if l != 2:
                big.append(l, k.cuda(), v.cuda())
            assert_close(big.decode_attention(l, q.cuda()).cpu().numpy(), ref)


def test_prefill_argument_checks():
    c = SharedKVCache(1, 2, 2, 128, 1, 64, "bf16")
    q = torch.zeros(1, 8, 2, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(KvsError) as e:          # nothing cached yet
        c.prefill_attention(0, q)
    assert e.value.status == kb.KVS_ERR_STATE
    k = torch.zeros(1, 4, 2, 128, dtype=torch.bfloat16, device="cuda")
    c.append(0, k, k)
    with pytest.raises(KvsError) as e:          # more queries than cached rows
        c.prefill_attention(0, q)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG
    f = SharedKVCache(1, 2, 2, 64, 1, 64, "f32")
    kk = torch.zeros(1, 4, 2, 64, dtype=torch.float32, device="cuda")
    f.append(0, kk, kk)
    with pytest.raises(KvsError) as e:          # fp32 storage has its own kernel; the checks are the same
        kb.kvs_prefill_attention(f.ctx, 0, torch.zeros(1, 8, 2, 64, device="cuda"), torch.zeros(1, 8, 2, 64, device="cuda"),
                                 1, 8, 0)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG
