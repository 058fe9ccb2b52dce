"""Parity of the CUDA path (through the C ABI) with the fp64 oracle on the same seeded inputs.

Bit-exact for indices, lengths and cached K/V; max-abs 2e-3 and relative-L2 1e-3 for
attention outputs (bf16 or fp32 inputs, fp32 accumulation).
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_2410_18517_b200 import KVS_OPT_EARLY_START, KVS_OPT_KERNEL, KVS_OPT_MAX_CTAS, KvsError, SharedKVCache
from paper_2410_18517_b200 import binding as kb
from paper_2410_18517_b200 import build as kbuild

from helpers import SampledRun, assert_close, make_cache, run_small

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


@pytest.fixture(autouse=True)
def _release_device_memory():
    yield
    import gc

    gc.collect()
    torch.cuda.empty_cache()


# ------------------------------------------------------------------ the tiny configuration, whole
def test_tiny_config_every_output_and_every_cached_bit():
    """L=4, 4 heads, D=64, B=2, 128 context rows, fp32, strategy {0,1,2,1}: one decode step and
    eight more, compared in full."""
    w = si.WORKLOADS["tiny"]
    cache, orc, worst = run_small(w, steps=9)
    assert cache.num_slots() == 3
    st = cache.stats()
    assert st["append_launches"] == 3 + 9 * 3 and st["append_skipped"] == 1 + 9
    assert st["attention_launches"] == 9 * 4 and st["combine_launches"] == 9 * 4
    assert [cache.seq_len(l) for l in range(4)] == [137] * 4
    assert worst[0] < 1e-4       # fp32 storage: far inside the bf16 tolerance


# ------------------------------------------------------------------ shapes, tails, strategies
SHAPES = [
    # dtype, D, Hq, Hkv
    ("bf16", 128, 4, 4), ("bf16", 128, 8, 2), ("bf16", 128, 4, 2), ("bf16", 128, 8, 1),
    ("bf16", 64, 4, 4), ("bf16", 64, 8, 2),
    ("f32", 64, 2, 2), ("f32", 128, 2, 2), ("f32", 128, 4, 1), ("f32", 128, 4, 2),
    # groups of eight q-heads with fp32 storage exist on the scalar kernel only (two passes of four heads)
    ("f32", 128, 8, 1), ("f32", 64, 8, 1), ("f32", 64, 16, 2),
]


@pytest.mark.parametrize("dtype,D,Hq,Hkv", SHAPES)
@pytest.mark.parametrize("context", [0, 63, 64, 65, 200, 1031])
def test_shapes_and_ragged_tails(dtype, D, Hq, Hkv, context):
    """Context lengths around the 32/64/128-row tile edges, 3 decode steps, chain strategy."""
    w = si.Workload(f"s_{dtype}_{D}_{Hq}_{Hkv}_{context}", L=4, Hq=Hq, Hkv=Hkv, D=D, B=3, context=context,
                    dtype=dtype, n_shared=0, map_seed=0, steps=3, fixed_map=(0, 0, 1, 2))
    cache, orc, _ = run_small(w, steps=3)
    assert cache.num_slots() == 1


@pytest.mark.parametrize("kernel", [1, 2])
@pytest.mark.parametrize("D,Hq,Hkv", [(128, 4, 4), (128, 4, 2), (128, 8, 2), (128, 8, 1), (64, 2, 2), (64, 4, 2),
                                      (64, 8, 2), (64, 8, 1)])
@pytest.mark.parametrize("context", [0, 15, 127, 128, 129, 700])
def test_both_kernels_on_every_group_size(kernel, D, Hq, Hkv, context):
    """bf16: the scalar and the tensor-core kernel, forced, on group sizes 1, 2, 4 and 8."""
    w = si.Workload(f"k{kernel}_{D}_{Hq}_{Hkv}_{context}", L=3, Hq=Hq, Hkv=Hkv, D=D, B=2, context=context,
                    dtype="bf16", n_shared=1, map_seed=0, steps=2, fixed_map=(0, 1, 0))
    cache, _, _ = run_small(w, steps=2, options=[(KVS_OPT_KERNEL, kernel)])
    assert cache.last_launch()["kernel"] == kernel


@pytest.mark.parametrize("G", [3, 5, 6, 7])
@pytest.mark.parametrize("D", [64, 128])
def test_group_sizes_that_are_not_powers_of_two(G, D):
    """48 q-heads over 8 kv-heads (InternLM2-20B's shape) is a group of 6: bf16 only, tensor-core kernel."""
    w = si.Workload(f"g{G}_{D}", L=3, Hq=2 * G, Hkv=2, D=D, B=2, context=333, dtype="bf16", n_shared=1, map_seed=0,
                    steps=2, fixed_map=(0, 1, 0))
    cache, _, _ = run_small(w, steps=2)
    assert cache.last_launch()["kernel"] == 2
    with pytest.raises(KvsError):
        cache.set_option(KVS_OPT_KERNEL, 1)           # the scalar kernel has groups of 1, 2, 4, 8 only


def test_auto_kernel_choice():
    """Groups of four or more bf16 q-heads go to the tensor cores; fp32 storage never does."""
    for Hq, Hkv, dtype, want in [(4, 4, "bf16", 1), (4, 2, "bf16", 1), (8, 2, "bf16", 2), (8, 1, "bf16", 2),
                                 (8, 2, "f32", 1)]:
        w = si.Workload(f"auto_{Hq}_{Hkv}_{dtype}", L=1, Hq=Hq, Hkv=Hkv, D=128, B=1, context=100, dtype=dtype,
                        n_shared=0, map_seed=0, steps=1)
        cache, _, _ = run_small(w, steps=1)
        assert cache.last_launch()["kernel"] == want
    with pytest.raises(KvsError):
        cache.set_option(KVS_OPT_KERNEL, 2)          # the last cache is fp32


@pytest.mark.parametrize("max_ctas", [1, 2, 5, 37, 0])
def test_tensor_core_kernel_any_split(max_ctas):
    w = si.Workload(f"mma_split_{max_ctas}", L=2, Hq=8, Hkv=2, D=128, B=2, context=1500, dtype="bf16",
                    n_shared=1, map_seed=0, steps=2, fixed_map=(0, 0))
    cache, _, _ = run_small(w, steps=2, options=[(KVS_OPT_MAX_CTAS, max_ctas), (KVS_OPT_KERNEL, 2)])
    assert cache.last_launch()["kernel"] == 2


@pytest.mark.parametrize("max_ctas", [1, 2, 5, 37, 0])
def test_any_split_of_the_tile_line_gives_the_same_answer(max_ctas):
    """The tile line of all units is cut at arbitrary places; results must not depend on it."""
    w = si.Workload(f"split_{max_ctas}", L=2, Hq=4, Hkv=4, D=128, B=2, context=1500, dtype="bf16",
                    n_shared=1, map_seed=0, steps=2, fixed_map=(0, 0))
    cache, _, _ = run_small(w, steps=2, options=[(KVS_OPT_MAX_CTAS, max_ctas)])
    if max_ctas:
        assert cache.last_launch()["ctas"] == max_ctas


@pytest.mark.parametrize("early", [0, 1])
@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (8, 2)])
def test_early_start_launches_change_nothing(early, Hq, Hkv):
    """Kernels that may start while their predecessor drains (and prefetch rows nothing in flight
    writes) against plain stream-ordered launches: same bits, and both match the oracle.  The
    context is appended immediately before the first step, 12 steps follow back to back."""
    w = si.Workload(f"early_{Hq}_{Hkv}", L=4, Hq=Hq, Hkv=Hkv, D=128, B=2, context=900, dtype="bf16", n_shared=2,
                    map_seed=0, steps=12, fixed_map=(0, 0, 2, 2))
    cache, _, _ = run_small(w, steps=12, options=[(KVS_OPT_EARLY_START, early)])
    ref_cache, _, _ = run_small(w, steps=12, options=[(KVS_OPT_EARLY_START, 0)], check_cache=False)
    q = si.step_qkv(w, 99, 1, device="cuda")[0]
    assert torch.equal(cache.decode_attention(1, q), ref_cache.decode_attention(1, q))


@pytest.mark.parametrize("case", range(24))
def test_random_small_configurations(case):
    """Seeded random layers / heads / group size / head size / type / batch / context / strategy
    (chains and fan-out included), a few decode steps, everything compared."""
    rng = np.random.default_rng(1000 + case)
    L = int(rng.integers(1, 7))
    Hkv = int(rng.choice([1, 2, 3, 4]))
    G = int(rng.choice([1, 2, 4, 8]))
    D = int(rng.choice([64, 128]))
    dtype = str(rng.choice(["bf16", "bf16", "f32"]))
    B = int(rng.integers(1, 5))
    context = int(rng.integers(0, 400))
    sm = tuple(int(rng.integers(0, l + 1)) if rng.random() < 0.5 else l for l in range(L))
    w = si.Workload(f"rand_{case}", L=L, Hq=Hkv * G, Hkv=Hkv, D=D, B=B, context=context, dtype=dtype, n_shared=0,
                    map_seed=0, steps=3, fixed_map=sm)
    opts = [(KVS_OPT_MAX_CTAS, int(rng.integers(1, 40)))] if rng.random() < 0.5 else []
    cache, orc, _ = run_small(w, steps=int(rng.integers(1, 4)), options=opts)
    n_slots, _, _ = oracle.slot_table(sm)
    assert cache.num_slots() == n_slots


def test_many_small_units_per_block():
    """More units than thread blocks and only a few tiles each: blocks span several whole units."""
    w = si.Workload("many_units", L=1, Hq=16, Hkv=16, D=128, B=40, context=130, dtype="bf16",
                    n_shared=0, map_seed=0, steps=1)
    run_small(w, steps=1)


def test_explicit_softmax_scale():
    w = si.Workload("scaled", L=1, Hq=2, Hkv=2, D=64, B=1, context=300, dtype="bf16", n_shared=0, map_seed=0, steps=1)
    run_small(w, steps=1, scale=0.2)


def test_smaller_batch_than_max_batch():
    w = si.Workload("subbatch", L=2, Hq=4, Hkv=2, D=128, B=2, context=100, dtype="bf16", n_shared=1, map_seed=0,
                    steps=1, fixed_map=(0, 0))
    cache = SharedKVCache(w.L, w.Hq, w.Hkv, w.D, 5, 256, "bf16", share_map=[0, 0])
    orc = oracle.Oracle(w.L, w.Hq, w.Hkv, w.D, w.B, [0, 0])
    k, v = si.context_kv(w, 0)
    cache.append(0, k.cuda(), v.cuda())
    orc.layer_forward(0, None, k.double().numpy(), v.double().numpy())
    for l in range(2):
        q, _, _ = si.step_qkv(w, 0, l)
        ref = orc.layer_forward(l, q.double().numpy())
        assert_close(cache.decode_attention(l, q.cuda()).cpu().numpy(), ref)
    with pytest.raises(KvsError) as e:      # more sequences than were cached
        cache.decode_attention(0, torch.zeros(3, 4, 128, dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == kb.KVS_ERR_INVALID_ARG


# ------------------------------------------------------------------ sharing semantics on the device
def test_append_on_sharing_layer_changes_no_byte_and_no_length():
    w = si.WORKLOADS["tiny"]
    cache = make_cache(w, 8)
    for l in range(w.L):
        k, v = si.context_kv(w, l)
        cache.append(l, k.cuda(), v.cuda())
    torch.cuda.synchronize()
    before = cache.pool.clone()
    lens = [cache.seq_len(l) for l in range(w.L)]
    launches = cache.stats()["append_launches"]
    _, k, v = si.step_qkv(w, 0, 3)
    cache.append(3, k.cuda(), v.cuda())        # layer 3 shares layer 1's cache
    cache.append(3, None, None, w.B, 5)        # pointers are not needed at all
    torch.cuda.synchronize()
    assert torch.equal(before, cache.pool)
    assert [cache.seq_len(l) for l in range(w.L)] == lens
    assert cache.stats()["append_launches"] == launches and cache.stats()["append_skipped"] == 3


def test_sharing_layer_sees_the_sources_newest_token():
    w = si.Workload("newest", L=2, Hq=2, Hkv=2, D=64, B=1, context=4, dtype="f32", n_shared=1, map_seed=0, steps=1,
                    fixed_map=(0, 0))
    cache = make_cache(w, 2)
    k, v = si.context_kv(w, 0)
    cache.append(0, k.cuda(), v.cuda())
    q = torch.zeros(1, 2, 64, device="cuda")
    knew = torch.zeros(1, 1, 2, 64, device="cuda")
    vnew = torch.full((1, 1, 2, 64), 100.0, device="cuda")
    cache.append(0, knew, vnew)
    out = cache.decode_attention(1, q)        # q = 0: uniform weights over 5 rows, the new one included
    ref = (v[0].double().sum(0) + 100.0) / 5.0
    np.testing.assert_allclose(out[0].cpu().numpy(), ref.numpy(), atol=1e-4)
    assert cache.seq_len(1) == 5


def test_error_paths_launch_nothing():
    w = si.WORKLOADS["tiny"]
    cache = make_cache(w, 0)               # capacity exactly 128
    q = torch.zeros(2, 4, 64, device="cuda")
    with pytest.raises(KvsError) as e:     # empty slot
        cache.decode_attention(0, q)
    assert e.value.status == kb.KVS_ERR_STATE
    k, v = si.context_kv(w, 0)
    cache.append(0, k.cuda(), v.cuda())
    _, k1, v1 = si.step_qkv(w, 0, 0)
    torch.cuda.synchronize()
    before = cache.pool.clone()
    with pytest.raises(KvsError) as e:     # 129th row
        cache.append(0, k1.cuda(), v1.cuda())
    assert e.value.status == kb.KVS_ERR_CAPACITY
    with pytest.raises(KvsError) as e:     # a different batch than the cached one
        cache.append(1, k1[:1].contiguous().cuda(), v1[:1].contiguous().cuda())
    assert e.value.status == kb.KVS_ERR_INVALID_ARG
    with pytest.raises(KvsError) as e:     # strategy is fixed once rows are cached
        kb.kvs_set_share_map(cache.ctx, [0, 0, 0, 0])
    assert e.value.status == kb.KVS_ERR_STATE
    with pytest.raises(KvsError):
        kb.kvs_append(cache.ctx, 1, None, None, 2, 1)
    # pointers that are not 16-byte aligned are refused (the kernels read 16-byte vectors)
    flat = torch.zeros(k1.numel() + 8, dtype=k1.dtype, device="cuda")
    k_off = flat[1 : 1 + k1.numel()].view(k1.shape)
    qflat = torch.zeros(q.numel() + 8, dtype=q.dtype, device="cuda")
    q_off = qflat[1 : 1 + q.numel()].view(q.shape)
    for call in (lambda: cache.append(1, k_off, k_off), lambda: cache.decode_attention(0, q_off),
                 lambda: cache.decode_step(1, q_off, v1.cuda(), v1.cuda()),
                 lambda: cache.decode_step(1, q, k_off, k_off)):
        with pytest.raises(KvsError) as e:
            call()
        assert e.value.status == kb.KVS_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert torch.equal(before, cache.pool) and cache.seq_len(0) == 128
    cache.reset()
    assert cache.seq_len(0) == 0
    kb.kvs_set_share_map(cache.ctx, [0, 0, 0, 0])
    assert cache.num_slots() == 1


def test_repeat_runs_are_bit_identical():
    w = si.Workload("det", L=1, Hq=8, Hkv=2, D=128, B=4, context=3000, dtype="bf16", n_shared=0, map_seed=0, steps=1)
    cache = make_cache(w, 1)
    k, v = si.context_kv(w, 0, device="cuda")
    cache.append(0, k, v)
    q = si.step_qkv(w, 0, 0, device="cuda")[0]
    a = cache.decode_attention(0, q).clone()
    for _ in range(3):
        assert torch.equal(a, cache.decode_attention(0, q))


@pytest.mark.parametrize("layers,chunks", [(4, None), (4, 1), (11, 1), (11, 2), (11, 3), (11, 4), (11, 8)])
def test_step_host_equals_per_layer_calls(layers, chunks):
    w = si.WORKLOADS["tiny"]
    if layers != w.L:
        w = w.scaled(L=layers, fixed_map=None, n_shared=3, map_seed=5)
    sm = w.share_map()
    n_own = int((sm == np.arange(w.L)).sum())
    a, b = make_cache(w, 4), make_cache(w, 4)
    if chunks is not None:
        a.set_option(kb.KVS_OPT_HOST_CHUNKS, chunks)
    for l in range(w.L):
        if sm[l] != l:
            continue
        k, v = si.context_kv(w, l)
        a.append(l, k.cuda(), v.cuda())
        b.append(l, k.cuda(), v.cuda())
    for t in range(3):
        qs, ks, vs = zip(*[si.step_qkv(w, t, l) for l in range(w.L)])
        qh, kh, vh = torch.stack(qs).pin_memory(), torch.stack(ks).pin_memory(), torch.stack(vs).pin_memory()
        oh = torch.empty(w.L, w.B, w.Hq, w.D, dtype=torch.float32).pin_memory()
        h2d, d2h = a.step_host(qh, kh, vh, oh)
        assert d2h == oh.numel() * 4
        assert h2d == qh.numel() * 4 + 2 * n_own * kh[0].numel() * 4      # K/V of the own-cache layers only
        for l in range(w.L):
            if sm[l] == l:
                b.append(l, ks[l].cuda(), vs[l].cuda())
            assert torch.equal(b.decode_attention(l, qs[l].cuda()).cpu(), oh[l])
    torch.cuda.synchronize()
    assert torch.equal(a.pool, b.pool)


@pytest.mark.parametrize("chunks", [1, 4])
def test_step_host_at_a_size_with_long_kernels(chunks):
    """Eight layers of the 7B shape at 2000 rows: every attention kernel runs for tens of
    microseconds, so a copy that did not wait for its kernel (or a kernel for its copy) would show.
    The whole-step call from host buffers must give the bits of the per-layer calls, outputs and
    cached rows, over three steps."""
    L, Hq, D, B, n = 8, 32, 128, 8, 2000
    w = si.Workload("host_big", L=L, Hq=Hq, Hkv=Hq, D=D, B=B, context=n, dtype="bf16", n_shared=2, map_seed=3, steps=3)
    sm = w.share_map()
    a, b = make_cache(w, 4), make_cache(w, 4)
    a.set_option(kb.KVS_OPT_HOST_CHUNKS, chunks)
    for l in range(L):
        if sm[l] != l:
            continue
        k, v = si.context_kv(w, l, device="cuda")
        a.append(l, k, v)
        b.append(l, k, v)
    for t in range(3):
        qs, ks, vs = zip(*[si.step_qkv(w, t, l) for l in range(L)])
        qh, kh, vh = torch.stack(qs).pin_memory(), torch.stack(ks).pin_memory(), torch.stack(vs).pin_memory()
        oh = torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32).pin_memory()
        a.step_host(qh, kh, vh, oh)
        for l in range(L):
            if sm[l] == l:
                b.append(l, ks[l].cuda(), vs[l].cuda())
            assert torch.equal(b.decode_attention(l, qs[l].cuda()).cpu(), oh[l]), (t, l)
    torch.cuda.synchronize()
    assert torch.equal(a.pool, b.pool) and a.device_status() == 0


def test_read_roof_checksum():
    x = torch.randint(0, 2**31 - 1, (3 * 32768 // 4 * 7,), dtype=torch.int32, device="cuda")
    chk = torch.zeros(1, dtype=torch.int64, device="cuda")
    kb.kvs_read_roof(x, x.numel() * 4, chk, 0, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    ref = np.bitwise_xor.reduce(x.cpu().numpy().view(np.uint32))
    assert int(chk.item()) == int(ref)


# ------------------------------------------------------------------ full-size configurations, sampled units
def test_7b_mha_full_size_sampled_units():
    """32 layers, 32 heads, D=128, B=8, 4096 context, bf16, 8 of 32 layers sharing: the
    benchmark's launch configuration; 64 sampled (layer, b, head) units incl. every sharing layer."""
    run = SampledRun(si.WORKLOADS["7b_mha"], steps=2, n_samples=64)
    assert run.cache.num_slots() == 24
    run.load_context()
    run.step(0, check=True)
    run.step(1, check=True)
    run.check_cached_rows()
    assert run.cache.device_status() == 0
    st = run.cache.stats()
    assert st["append_launches"] == 24 * 3 and st["append_skipped"] == 8 * 3
    assert st["kv_bytes_read"] == sum(2 * 8 * 32 * n * 256 for n in (4097, 4098)) * 32


def test_gqa_long_full_size_sampled_units():
    """32 q-heads over 8 kv-heads, B=4, 32768 context, 10 of 32 layers sharing."""
    run = SampledRun(si.WORKLOADS["gqa_long"], steps=1, n_samples=48)
    assert run.cache.num_slots() == 22
    run.load_context()
    run.step(0, check=True)
    run.check_cached_rows()
    assert run.cache.device_status() == 0


def test_13b_mha_64_steps_sampled_units():
    """40 layers, 40 heads, B=16, 8192 context, 12 of 40 sharing, 64 consecutive steps with appends;
    sampled units checked at steps 1, 32 and 64, appended rows bit-exact."""
    run = SampledRun(si.WORKLOADS["13b_mha"], steps=64, n_samples=52)
    assert run.cache.num_slots() == 28
    run.load_context()
    for t in range(64):
        run.step(t, check=(t in (0, 31, 63)))
    run.check_cached_rows()
    assert [run.cache.seq_len(l) for l in range(40)] == [8192 + 64] * 40
    assert run.cache.device_status() == 0


# ------------------------------------------------------------------ units finished inside the split-K kernel
@pytest.mark.parametrize("Hq,Hkv,B,dtype,kernel", [(8, 8, 24, "bf16", 0), (16, 4, 40, "bf16", 0), (8, 4, 80, "bf16", 1),
                                                   (4, 4, 40, "f32", 0), (8, 1, 160, "bf16", 0)])
@pytest.mark.parametrize("context", [40, 129, 700])
def test_units_finished_inside_the_split_k_kernel(Hq, Hkv, B, dtype, kernel, context):
    """At least as many (sequence, kv-head) units as thread blocks: no combine launch, the block that
    holds a unit's first piece merges it with the second.  Every output against the oracle, the same
    bits with the separate combine kernel forced, and again on a second run."""
    from paper_2410_18517_b200 import KVS_OPT_FINISH_IN_KERNEL

    w = si.Workload(f"fin_{Hq}_{Hkv}_{B}_{dtype}_{context}", L=2, Hq=Hq, Hkv=Hkv, D=128, B=B, context=context,
                    dtype=dtype, n_shared=1, map_seed=0, steps=2, fixed_map=(0, 0))
    opts = [(KVS_OPT_KERNEL, kernel)] if kernel else []
    cache, _, _ = run_small(w, steps=2, options=opts, use_step=True)
    st = cache.stats()
    assert st["combine_launches"] == 0 and st["attention_launches"] == 4
    two, _, _ = run_small(w, steps=2, options=opts + [(KVS_OPT_FINISH_IN_KERNEL, 0)], use_step=True, check_cache=False)
    assert two.stats()["combine_launches"] == 4
    q = si.step_qkv(w, 7, 1, device="cuda")[0]
    a, b = cache.decode_attention(1, q), cache.decode_attention(1, q)
    assert torch.equal(a, b)
    c = two.decode_attention(1, q)
    err = (a - c).abs().max().item()
    assert err <= 1e-5, err          # same pieces, merged in the same order by different code: rounding only
    assert cache.device_status() == 0


@pytest.mark.parametrize("Hq,Hkv,B,context,dtype", [(32, 8, 32, 1024, "bf16"), (32, 32, 8, 4096, "bf16"), (8, 1, 160, 129, "bf16"),
                                                   (4, 4, 40, 700, "f32"), (32, 8, 8, 8192, "bf16")])
def test_launches_back_to_back_give_the_same_bits(Hq, Hkv, B, context, dtype):
    """Hundreds of launches queued without a pause, each starting early beside the one before: the hand-over
    flags and partial results of one launch must be gone before the next uses them.  Same inputs, so the same
    bits every time; then decode steps (the append rides in the kernel) twice from the same cache length."""
    reps = 100
    w = si.Workload(f"b2b_{Hq}_{Hkv}_{B}_{context}", L=4, Hq=Hq, Hkv=Hkv, D=128, B=B, context=context, dtype=dtype,
                    n_shared=1, map_seed=0, steps=1, fixed_map=(0, 1, 2, 0))
    cache = make_cache(w, reps + 8)
    for l in range(3):
        k, v = si.context_kv(w, l, device="cuda")
        cache.append(l, k, v)
    ins = [si.step_qkv(w, 0, l, device="cuda") for l in range(4)]
    outs = [[torch.empty(B, Hq, 128, device="cuda") for _ in range(4)] for _ in range(reps)]
    torch.cuda.synchronize()
    for r in range(reps):
        for l in range(4):
            cache.decode_attention(l, ins[l][0], out=outs[r][l])
    torch.cuda.synchronize()
    assert all(torch.equal(outs[r][l], outs[0][l]) for r in range(1, reps) for l in range(4))
    assert not torch.equal(outs[0][0], outs[0][3]) and cache.device_status() == 0     # layer 3 reads slot 0 with its own q
    runs = []
    for _ in range(2):
        cache.truncate(context)
        res = []
        for r in range(32):
            for l in range(4):
                q, k, v = ins[l]
                own = l < 3
                res.append(cache.decode_step(l, q, k if own else None, v if own else None))
        torch.cuda.synchronize()
        runs.append(res)
    assert all(torch.equal(a, b) for a, b in zip(*runs))
    assert cache.device_status() == 0


# ------------------------------------------------------------------ sweep points at full size
@pytest.mark.parametrize("name", ["sweep_b32_n1024_p10", "sweep_b64_n1024_p4", "sweep_b32_n8192_p8"])
def test_sweep_points_sampled_units(name):
    """32 q-heads over 8 kv-heads at batch 32 and 64 (more units than thread blocks: the tensor-core kernel
    finishes the units itself), in the launch configuration the sweep and the benchmark time."""
    w = si.workload_by_name(name)
    run = SampledRun(w, steps=2, n_samples=w.n_shared + 24, seed=3)
    run.load_context()
    for t in range(2):
        run.step(t, check=True)
    run.check_cached_rows()
    assert run.cache.last_launch()["kernel"] == 2 and run.cache.stats()["combine_launches"] == 0
    assert run.cache.device_status() == 0
