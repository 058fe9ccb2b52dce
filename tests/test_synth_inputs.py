"""The seeded input generators: share maps obey the stated recipe, tensors are reproducible."""
import numpy as np
import torch

import synth_inputs as si


def test_random_share_map_recipe():
    for L, P in [(32, 8), (40, 12), (32, 10), (32, 4), (32, 0), (80, 20), (4, 2)]:
        for seed in range(5):
            sm = si.random_share_map(L, P, seed)
            targets = [l for l in range(L) if sm[l] != l]
            sources = [int(sm[t]) for t in targets]
            assert len(targets) == P and sm[0] == 0
            assert all(s < t for s, t in zip(sources, targets))
            assert len(set(sources)) == P                      # distinct sources
            assert all(sm[s] == s for s in sources)            # that compute their own cache
            np.testing.assert_array_equal(sm, si.random_share_map(L, P, seed))


def test_named_workloads_match_their_descriptions():
    w = si.WORKLOADS
    assert list(w["tiny"].share_map()) == [0, 1, 2, 1]
    assert (w["7b_mha"].L, w["7b_mha"].Hq, w["7b_mha"].Hkv, w["7b_mha"].B, w["7b_mha"].context) == (32, 32, 32, 8, 4096)
    assert sum(w["7b_mha"].share_map() != np.arange(32)) == 8
    assert sum(w["13b_mha"].share_map() != np.arange(40)) == 12
    assert sum(w["gqa_long"].share_map() != np.arange(32)) == 10 and w["gqa_long"].G == 4
    assert w["7b_mha"].kv_read_bytes_per_layer(4096) == 512 * 2**20
    assert w["13b_mha"].kv_read_bytes_per_layer(8192) == 2560 * 2**20
    assert len(si.sweep_points()) == 48


def test_tensors_are_seeded_and_rounded_to_storage_type():
    w = si.WORKLOADS["tiny"]
    q1, k1, v1 = si.step_qkv(w, 3, 2)
    q2, k2, v2 = si.step_qkv(w, 3, 2)
    assert torch.equal(q1, q2) and torch.equal(k1, k2) and torch.equal(v1, v2)
    assert not torch.equal(q1, si.step_qkv(w, 4, 2)[0])
    assert q1.dtype == torch.float32 and q1.shape == (2, 4, 64) and k1.shape == (2, 1, 4, 64)
    wb = w.scaled(dtype="bf16")
    assert si.step_qkv(wb, 0, 0)[0].dtype == torch.bfloat16
    k, v = si.context_kv(w, 1)
    assert k.shape == (2, 128, 4, 64) and abs(float(k.mean())) < 0.02 and abs(float(k.std()) - 1) < 0.02


def test_batch_sharding_covers_the_batch_once():
    for B in (1, 7, 8, 64):
        for ws in (1, 2, 3, 8):
            spans = [si.shard_batch(B, ws, r) for r in range(ws)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(spans[:-1], spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
