"""The strategy-search reductions on the GPU (layer-pair KV distances, mean-representation cosine)
against the fp64 oracle.  fp32 accumulation over up to millions of terms: relative 2e-4."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_2410_18517_b200 import KvsError, SharedKVCache
from paper_2410_18517_b200 import binding as kb
from paper_2410_18517_b200 import build as kbuild

pytestmark = pytest.mark.gpu
REL = 2e-4


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


def _load_both(L, Hq, Hkv, D, B, n, dtype, share_map, max_batch=None):
    w = si.Workload(f"search_{L}_{Hkv}_{D}_{B}_{n}_{dtype}", L=L, Hq=Hq, Hkv=Hkv, D=D, B=B, context=n, dtype=dtype,
                    n_shared=0, map_seed=0, steps=0)
    cache = SharedKVCache(L, Hq, Hkv, D, max_batch or B, n, dtype, share_map=share_map)
    orc = oracle.Oracle(L, Hq, Hkv, D, B, share_map)
    for l in range(L):
        k, v = si.context_kv(w, l)
        if l % 3 == 2:                              # make some layers close to each other
            k0, v0 = si.context_kv(w, l - 1)
            k, v = (k0.float() + 0.05 * k.float()).to(k.dtype), (v0.float() + 0.05 * v.float()).to(v.dtype)
        orc.layer_forward(l, None, k.double().numpy(), v.double().numpy())
        if share_map[l] == l:
            cache.append(l, k.cuda(), v.cuda())
    return cache, orc


@pytest.mark.parametrize("L,Hq,Hkv,D,B,n,dtype", [
    (6, 4, 2, 64, 5, 37, "bf16"), (6, 4, 2, 128, 3, 64, "f32"), (5, 2, 1, 128, 7, 129, "bf16"),
    (32, 8, 8, 128, 6, 64, "bf16"), (40, 4, 2, 64, 4, 33, "bf16"), (80, 2, 1, 64, 2, 16, "bf16"),
    (8, 4, 4, 128, 3, 600, "bf16"), (5, 2, 2, 128, 2, 1100, "f32")])     # the last two: several chunks per thread block
def test_layer_distances(L, Hq, Hkv, D, B, n, dtype):
    sm = list(range(L))
    sm[L - 1] = 1                                   # one sharing layer: it has layer 1's cache
    cache, orc = _load_both(L, Hq, Hkv, D, B, n, dtype, sm, max_batch=B + 1)
    ref = orc.layer_distances()
    # the oracle's sharing layer gets its literal copy at its turn (done in _load_both's layer_forward)
    got = cache.layer_distances(B).double().cpu().numpy()
    assert np.all(np.diag(got) == 0) and np.array_equal(got, got.T)
    assert got[L - 1, 1] == 0.0
    np.testing.assert_allclose(got, ref, rtol=REL, atol=1e-6)
    # the search ranks pairs by distance, descending: same order wherever the oracle's gap is clear
    iu = np.triu_indices(L, 1)
    order_ref, order_got = np.argsort(-ref[iu], kind="stable"), np.argsort(-got[iu], kind="stable")
    sorted_ref = ref[iu][order_ref]
    clear = np.abs(np.diff(sorted_ref)) > 4 * REL * sorted_ref[:-1]       # gap k | k+1 is unambiguous
    isolated = np.append(clear, True) & np.append(True, clear)             # both neighbours clearly apart
    assert np.array_equal(order_ref[isolated], order_got[isolated])
    assert cache.device_status() == 0 and cache.stats()["search_launches"] >= 3


def test_layer_distances_state_errors():
    cache = SharedKVCache(2, 2, 2, 64, 2, 32, "bf16")
    d = torch.empty(2, 2, device="cuda")
    with pytest.raises(KvsError) as e:
        kb.kvs_layer_distances(cache.ctx, 2, d, 0)
    assert e.value.status == kb.KVS_ERR_STATE                      # nothing cached
    k = torch.randn(2, 8, 2, 64, device="cuda").bfloat16()
    cache.append(0, k, k)
    with pytest.raises(KvsError) as e:
        kb.kvs_layer_distances(cache.ctx, 2, d, 0)
    assert e.value.status == kb.KVS_ERR_STATE                      # layer 1 is still empty
    cache.append(1, k, k)
    with pytest.raises(KvsError) as e:
        kb.kvs_layer_distances(cache.ctx, 3, d, 0)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG                # more samples than cached
    kb.kvs_layer_distances(cache.ctx, 2, d, 0)
    assert float(d[0, 1]) == 0.0                                   # both layers hold the same rows
    # a stream that is being captured is refused (the call is not meant for graphs); the capture survives
    side, graph = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    marker = torch.zeros(4, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        with pytest.raises(KvsError) as e:
            kb.kvs_layer_distances(cache.ctx, 2, d, side.cuda_stream)
        marker += 1.0
    assert e.value.status == kb.KVS_ERR_STATE
    graph.replay()
    torch.cuda.synchronize()
    assert float(marker[0]) == 1.0


@pytest.mark.parametrize("S,dim,dtype", [(30, 4096, "bf16"), (3, 10, "f32"), (7, 64 * 5120, "bf16"),
                                          (3, 3 * 1024 * 1024, "bf16"), (2, 1024 * 1024 + 6, "f32")])   # several passes per block
def test_mean_cosine(S, dim, dtype):
    cache = SharedKVCache(1, 1, 1, 64, 1, 8, dtype)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    a = si.normal((1, "cos_a", S, dim), (S, dim), td)
    b = (0.6 * a.float() + 0.8 * si.normal((1, "cos_b", S, dim), (S, dim), torch.float32)).to(td)
    ref = oracle.mean_cosine(a.double().numpy(), b.double().numpy())
    got = float(cache.mean_cosine(a.cuda(), b.cuda()).item())
    assert abs(got - ref) < 2e-5
    assert abs(float(cache.mean_cosine(a.cuda(), a.cuda()).item()) - 1.0) < 1e-5
    with pytest.raises(KvsError):
        kb.kvs_mean_cosine(cache.ctx, a.cuda(), b.cuda(), S, 3, torch.empty(1, device="cuda"), 0)   # odd dim
