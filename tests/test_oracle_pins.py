"""Pins for the fp64 CPU oracle: it is checked against things other than itself.

* a library routine: torch's scaled_dot_product_attention in float64, which the
  identity share map must reproduce (ordinary per-layer attention);
* brute force: an independent few-line numpy expression on tiny shapes, with
  sharing applied by index arithmetic instead of the oracle's literal copy;
* closed forms and invariances of softmax attention;
* the invariants of layer sharing (own Q over the source's K/V; number of
  caches = layers - shared layers, on the layer counts the paper prints);
* the split/combine identity of the softmax sum.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from synth_inputs import random_share_map

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(12345)


def brute_attention(q, K, V):
    """softmax(q K^T / sqrt(D)) V with an explicit n x 1 score vector (numpy, fp64)."""
    sc = (K @ q.reshape(-1, 1)) / np.sqrt(q.shape[0])           # [n, 1]
    w = np.exp(sc - sc.max())
    w = w / w.sum()
    return (w * V).sum(axis=0)


def run_oracle(L, Hq, Hkv, D, B, share_map, ctx, steps, rng):
    """Load ``ctx`` rows, then ``steps`` decode steps.  Returns inputs and outputs."""
    o = oracle.Oracle(L, Hq, Hkv, D, B, share_map)
    kc = rng.standard_normal((L, B, ctx, Hkv, D))
    vc = rng.standard_normal((L, B, ctx, Hkv, D))
    for l in range(L):
        o.layer_forward(l, None, kc[l], vc[l])
    qs = rng.standard_normal((steps, L, B, Hq, D))
    ks = rng.standard_normal((steps, L, B, 1, Hkv, D))
    vs = rng.standard_normal((steps, L, B, 1, Hkv, D))
    outs = np.stack([o.step(qs[t], ks[t], vs[t]) for t in range(steps)])
    return o, kc, vc, qs, ks, vs, outs


# ---------------------------------------------------------------- library pin
@pytest.mark.parametrize("Hq,Hkv,D,n", [(4, 4, 16, 37), (8, 2, 32, 65), (6, 3, 8, 5), (4, 1, 64, 129)])
def test_identity_map_equals_torch_sdpa_fp64(Hq, Hkv, D, n):
    L, B = 3, 2
    rng = np.random.default_rng(7)
    o, kc, vc, qs, ks, vs, outs = run_oracle(L, Hq, Hkv, D, B, np.arange(L), n - 1, 1, rng)
    G = Hq // Hkv
    for l in range(L):
        K = np.concatenate([kc[l], ks[0, l]], axis=1)            # [B][n][Hkv][D]
        V = np.concatenate([vc[l], vs[0, l]], axis=1)
        Kt = torch.from_numpy(K).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)   # [B][Hq][n][D]
        Vt = torch.from_numpy(V).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
        qt = torch.from_numpy(qs[0, l]).unsqueeze(2)             # [B][Hq][1][D]
        ref = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt).squeeze(2).numpy()
        np.testing.assert_allclose(outs[0, l], ref, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("share_map", [[0, 1, 2, 1], [0, 0, 0, 0], [0, 0, 1, 2], [0, 1, 1, 3], [0, 1, 2, 3]])
@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (4, 2), (3, 1)])
def test_brute_force_with_sharing(share_map, Hq, Hkv):
    """Sharing by index: layer l attends over the rows its *root* layer was given.

    Chains ([0,0,1,2]: 3 <- 2 <- 1 <- 0) must end at the layer that computes its own
    cache, and the root's row of the *current* step must be visible to the sharer.
    """
    L, D, B, ctx, steps = 4, 8, 2, 6, 3
    rng = np.random.default_rng(hash((tuple(share_map), Hq, Hkv)) % (2**32))
    o, kc, vc, qs, ks, vs, outs = run_oracle(L, Hq, Hkv, D, B, share_map, ctx, steps, rng)
    G = Hq // Hkv
    for t in range(steps):
        for l in range(L):
            r = l
            while share_map[r] != r:
                r = share_map[r]
            K = np.concatenate([kc[r]] + [ks[u, r] for u in range(t + 1)], axis=1)   # [B][n][Hkv][D]
            V = np.concatenate([vc[r]] + [vs[u, r] for u in range(t + 1)], axis=1)
            assert K.shape[1] == ctx + t + 1
            for b in range(B):
                for hq in range(Hq):
                    ref = brute_attention(qs[t, l, b, hq], K[b, :, hq // G], V[b, :, hq // G])
                    np.testing.assert_allclose(outs[t, l, b, hq], ref, rtol=0, atol=1e-13)


def test_unit_entry_points_agree_with_brute_force():
    rng = np.random.default_rng(3)
    U, n, D = 5, 23, 16
    q, K, V = rng.standard_normal((U, D)), rng.standard_normal((U, n, D)), rng.standard_normal((U, n, D))
    many = oracle.attend_units(q, K, V)
    for u in range(U):
        ref = brute_attention(q[u], K[u], V[u])
        np.testing.assert_allclose(oracle.attend_unit(q[u], K[u], V[u]), ref, atol=1e-13)
        np.testing.assert_allclose(many[u], ref, atol=1e-13)


def test_explicit_scale_is_used():
    rng = np.random.default_rng(4)
    n, D = 9, 8
    q, K, V = rng.standard_normal(D), rng.standard_normal((n, D)), rng.standard_normal((n, D))
    # scale s on q.K equals the default scale applied to q * s * sqrt(D)
    np.testing.assert_allclose(oracle.attend_unit(q, K, V, scale=0.37),
                               brute_attention(q * 0.37 * np.sqrt(D), K, V), atol=1e-13)


# ---------------------------------------------------------------- closed forms
def test_single_row_returns_that_value_row():
    q, K, V = RNG.standard_normal(8), RNG.standard_normal((1, 8)), RNG.standard_normal((1, 8))
    np.testing.assert_array_equal(oracle.attend_unit(q, K, V), V[0])


def test_equal_keys_or_zero_query_give_mean_of_values():
    n, D = 17, 8
    V = RNG.standard_normal((n, D))
    K = np.tile(RNG.standard_normal((1, D)), (n, 1))
    np.testing.assert_allclose(oracle.attend_unit(RNG.standard_normal(D), K, V), V.mean(0), atol=1e-14)
    np.testing.assert_allclose(oracle.attend_unit(np.zeros(D), RNG.standard_normal((n, D)), V),
                               V.mean(0), atol=1e-14)


def test_constant_values_are_returned():
    n, D = 11, 8
    c = RNG.standard_normal(D)
    out = oracle.attend_unit(RNG.standard_normal(D), RNG.standard_normal((n, D)), np.tile(c, (n, 1)))
    np.testing.assert_allclose(out, c, atol=1e-14)


def test_dominant_key_selects_its_value_row():
    n, D = 13, 8
    q = RNG.standard_normal(D)
    K = RNG.standard_normal((n, D)) * 0.1
    V = RNG.standard_normal((n, D))
    K[5] = q * (60.0 * np.sqrt(D) / (q @ q))       # score of row 5 is 60, the others are O(1)
    np.testing.assert_allclose(oracle.attend_unit(q, K, V), V[5], atol=1e-15 * 1e3)


def test_two_row_logistic_closed_form():
    """n = 2: weights are the logistic function of the score difference."""
    D = 4
    q, K, V = RNG.standard_normal(D), RNG.standard_normal((2, D)), RNG.standard_normal((2, D))
    delta = (q @ K[0] - q @ K[1]) / np.sqrt(D)
    w0 = 1.0 / (1.0 + np.exp(-delta))
    np.testing.assert_allclose(oracle.attend_unit(q, K, V), w0 * V[0] + (1 - w0) * V[1], atol=1e-14)


def test_row_permutation_invariance():
    n, D = 19, 8
    q, K, V = RNG.standard_normal(D), RNG.standard_normal((n, D)), RNG.standard_normal((n, D))
    perm = RNG.permutation(n)
    np.testing.assert_allclose(oracle.attend_unit(q, K[perm], V[perm]), oracle.attend_unit(q, K, V), atol=1e-14)


def test_softmax_shift_invariance():
    """Adding u to q changes every score by the same amount when all K_j.u are equal."""
    n, D = 15, 8
    q, V = RNG.standard_normal(D), RNG.standard_normal((n, D))
    K = RNG.standard_normal((n, D))
    u = np.zeros(D)
    u[0] = 3.0
    K[:, 0] = 0.7                                   # K_j . u = 2.1 for every row
    np.testing.assert_allclose(oracle.attend_unit(q + u, K, V), oracle.attend_unit(q, K, V), atol=1e-13)


def test_output_is_convex_combination_of_value_rows():
    n, D = 31, 8
    q, K, V = RNG.standard_normal(D), RNG.standard_normal((n, D)), RNG.standard_normal((n, D))
    out = oracle.attend_unit(q, K, V)
    assert np.all(out <= V.max(0) + 1e-14) and np.all(out >= V.min(0) - 1e-14)


# ---------------------------------------------------------------- sharing invariants
def test_sharing_layer_equals_own_query_over_source_kv():
    """Run the strategy [0,1,2,1]; then an unshared model whose layer-3 K/V inputs are layer 1's."""
    L, Hq, Hkv, D, B, ctx, steps = 4, 4, 2, 8, 2, 10, 4
    sm = [0, 1, 2, 1]
    rng = np.random.default_rng(11)
    _, kc, vc, qs, ks, vs, outs = run_oracle(L, Hq, Hkv, D, B, sm, ctx, steps, rng)
    kc2, vc2, ks2, vs2 = kc.copy(), vc.copy(), ks.copy(), vs.copy()
    kc2[3], vc2[3], ks2[:, 3], vs2[:, 3] = kc[1], vc[1], ks[:, 1], vs[:, 1]
    plain = oracle.Oracle(L, Hq, Hkv, D, B, np.arange(L))
    for l in range(L):
        plain.layer_forward(l, None, kc2[l], vc2[l])
    outs2 = np.stack([plain.step(qs[t], ks2[t], vs2[t]) for t in range(steps)])
    np.testing.assert_array_equal(outs, outs2)
    # and the sharing layer really differs from what its own K/V inputs would have given
    plain_own = oracle.Oracle(L, Hq, Hkv, D, B, np.arange(L))
    for l in range(L):
        plain_own.layer_forward(l, None, kc[l], vc[l])
    own = plain_own.step(qs[0], ks[0], vs[0])
    assert np.abs(own[3] - outs[0, 3]).max() > 1e-3
    np.testing.assert_array_equal(own[:3], outs[0, :3])


def test_sharing_layer_appends_nothing_and_mirrors_source():
    L, Hq, Hkv, D, B = 4, 2, 2, 4, 1
    sm = [0, 1, 2, 1]
    rng = np.random.default_rng(5)
    o, kc, vc, qs, ks, vs, outs = run_oracle(L, Hq, Hkv, D, B, sm, 3, 2, rng)
    assert [o.length(l) for l in range(L)] == [5, 5, 5, 5]
    K1, V1 = o.cache(1)
    K3, V3 = o.cache(3)
    np.testing.assert_array_equal(K1, K3)
    np.testing.assert_array_equal(V1, V3)
    # the rows handed to the sharing layer itself were never stored anywhere
    for l in range(L):
        K, _ = o.cache(l)
        assert not np.isin(ks[:, 3].ravel(), K.ravel()).any()
    # an own-cache layer stores exactly what it was given, in order, as [B][Hkv][n][D]
    K2, V2 = o.cache(2)
    exp = np.concatenate([kc[2], ks[0, 2], ks[1, 2]], axis=1).transpose(0, 2, 1, 3)
    np.testing.assert_array_equal(K2, exp)


def test_cache_update_only_call_on_sharing_layer_ignores_inputs():
    o = oracle.Oracle(2, 1, 1, 4, 1, [0, 0])
    k = RNG.standard_normal((1, 3, 1, 4))
    o.layer_forward(0, None, k, k)
    o.layer_forward(1, None, None, None)
    assert o.length(1) == 3
    o.layer_forward(1, None, RNG.standard_normal((1, 2, 1, 4)), RNG.standard_normal((1, 2, 1, 4)))
    assert o.length(1) == 3 and o.length(0) == 3


def _paper_layer_counts():
    rows = []
    with open(os.path.join(GOLDEN, "paper_layer_counts.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = line.split()
            rows.append((parts[0], int(parts[1]), [int(x) for x in parts[2:]]))
    return rows


@pytest.mark.parametrize("model,L,computed", _paper_layer_counts())
def test_cache_count_matches_paper_layer_column(model, L, computed):
    """The paper's tables list how many layers still compute a cache; that is L - #shared."""
    rates = [0.125, 0.25, 0.375]
    for i, c in enumerate(computed):
        P = L - c
        assert P == round(L * rates[i])              # Section 4.2 rates
        for seed in range(3):
            sm = random_share_map(L, P, seed)
            n, root, slot = oracle.slot_table(sm)
            assert n == c
            assert sorted(set(slot.tolist())) == list(range(c))
            assert all(sm[r] == r for r in root)


def test_slot_table_against_python_definition():
    rng = np.random.default_rng(0)
    for _ in range(200):
        L = int(rng.integers(1, 12))
        sm = np.array([int(rng.integers(0, l + 1)) for l in range(L)], dtype=np.int32)
        n, root, slot = oracle.slot_table(sm)
        roots = [l for l in range(L) if sm[l] == l]
        assert n == len(roots)
        for l in range(L):
            r = l
            while sm[r] != r:
                r = int(sm[r])
            assert root[l] == r and slot[l] == roots.index(r)


def test_illegal_strategies_are_rejected():
    assert oracle.slot_table([0, 2, 2]) is None       # source nearer the output than its target
    assert oracle.slot_table([1, 1]) is None          # layer 0 has no earlier layer
    assert oracle.slot_table([0, -1]) is None
    with pytest.raises(ValueError):
        oracle.Oracle(3, 2, 2, 4, 1, [0, 2, 2])
    with pytest.raises(ValueError):
        oracle.Oracle(2, 3, 2, 4, 1, [0, 1])          # 3 q-heads over 2 kv-heads


def test_empty_cache_is_an_error():
    o = oracle.Oracle(1, 1, 1, 4, 1, [0])
    with pytest.raises(RuntimeError):
        o.layer_forward(0, np.zeros((1, 1, 4)))


# ---------------------------------------------------------------- split / combine
@pytest.mark.parametrize("cuts", [[0, 40], [0, 1, 40], [0, 13, 14, 39, 40], list(range(0, 41, 8)), list(range(41))])
def test_any_row_partition_recombines_to_the_unsplit_result(cuts):
    n, D = 40, 16
    rng = np.random.default_rng(9)
    q, K, V = rng.standard_normal(D) * 3, rng.standard_normal((n, D)), rng.standard_normal((n, D))
    parts = [oracle.partial_unit(q, K, V, a, b) for a, b in zip(cuts[:-1], cuts[1:])]
    out = oracle.combine_partials(np.stack([p[0] for p in parts]), [p[1] for p in parts], [p[2] for p in parts])
    np.testing.assert_allclose(out, brute_attention(q, K, V), atol=1e-13)


def test_partial_of_everything_is_unnormalised_attention():
    n, D = 12, 8
    q, K, V = RNG.standard_normal(D), RNG.standard_normal((n, D)), RNG.standard_normal((n, D))
    o, m, l = oracle.partial_unit(q, K, V, 0, n)
    sc = K @ q / np.sqrt(D)
    assert m == pytest.approx(sc.max(), abs=1e-15)
    assert l == pytest.approx(np.exp(sc - sc.max()).sum(), abs=1e-13)
    np.testing.assert_allclose(o / l, brute_attention(q, K, V), atol=1e-14)


# ---------------------------------------------------------------- a planted mistake is caught
def test_pins_would_catch_a_transposed_group_mapping():
    """hq % Hkv instead of hq // G is a plausible slip; the SDPA pin must see it."""
    Hq, Hkv, D, n = 4, 2, 8, 7
    rng = np.random.default_rng(21)
    q, K, V = rng.standard_normal((Hq, D)), rng.standard_normal((Hkv, n, D)), rng.standard_normal((Hkv, n, D))
    right = np.stack([brute_attention(q[h], K[h // 2], V[h // 2]) for h in range(Hq)])
    wrong = np.stack([brute_attention(q[h], K[h % 2], V[h % 2]) for h in range(Hq)])
    o = oracle.Oracle(1, Hq, Hkv, D, 1, [0])
    got = o.layer_forward(0, q[None], K.transpose(1, 0, 2)[None], V.transpose(1, 0, 2)[None])[0]
    np.testing.assert_allclose(got, right, atol=1e-13)
    assert np.abs(got - wrong).max() > 1e-2


# ---------------------------------------------------------------- prefill (causal, many queries)
@pytest.mark.parametrize("Hq,Hkv,D,T", [(4, 4, 16, 33), (8, 2, 32, 17), (4, 1, 8, 64)])
def test_prefill_identity_map_equals_torch_causal_sdpa_fp64(Hq, Hkv, D, T):
    L, B = 2, 2
    rng = np.random.default_rng(31)
    o = oracle.Oracle(L, Hq, Hkv, D, B, np.arange(L))
    G = Hq // Hkv
    for l in range(L):
        q = rng.standard_normal((B, T, Hq, D))
        k = rng.standard_normal((B, T, Hkv, D))
        v = rng.standard_normal((B, T, Hkv, D))
        out = o.layer_prefill(l, q, k, v)
        qt = torch.from_numpy(q).permute(0, 2, 1, 3)
        kt = torch.from_numpy(k).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
        vt = torch.from_numpy(v).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
        ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True).permute(0, 2, 1, 3).numpy()
        np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("share_map", [[0, 1, 2, 1], [0, 0, 1, 2], [0, 1, 2, 3]])
def test_prefill_chunks_with_sharing_against_brute_force(share_map):
    """Two prompt chunks (5 rows, then 7): a query sees everything cached before its chunk plus its
    chunk up to itself; a sharing layer uses its root layer's rows, current chunk included."""
    L, Hq, Hkv, D, B = 4, 4, 2, 8, 2
    rng = np.random.default_rng(hash(tuple(share_map)) % (2**32))
    o = oracle.Oracle(L, Hq, Hkv, D, B, share_map)
    G = Hq // Hkv
    ks = [[rng.standard_normal((B, T, Hkv, D)) for T in (5, 7)] for _ in range(L)]
    vs = [[rng.standard_normal((B, T, Hkv, D)) for T in (5, 7)] for _ in range(L)]
    for c, T in enumerate((5, 7)):
        for l in range(L):
            q = rng.standard_normal((B, T, Hq, D))
            out = o.layer_prefill(l, q, ks[l][c], vs[l][c])
            r = l
            while share_map[r] != r:
                r = share_map[r]
            K = np.concatenate(ks[r][: c + 1], axis=1)
            V = np.concatenate(vs[r][: c + 1], axis=1)
            n = K.shape[1]
            for b in range(B):
                for i in range(T):
                    for hq in range(Hq):
                        lim = n - T + i + 1
                        ref = brute_attention(q[b, i, hq], K[b, :lim, hq // G], V[b, :lim, hq // G])
                        np.testing.assert_allclose(out[b, i, hq], ref, atol=1e-13)


def test_prefill_first_query_of_an_empty_cache_returns_first_value_row_and_one_query_is_decode():
    o = oracle.Oracle(1, 2, 2, 4, 1, [0])
    k, v, q = (RNG.standard_normal((1, 6, 2, 4)) for _ in range(3))
    out = o.layer_prefill(0, q, k, v)
    np.testing.assert_array_equal(out[0, 0], v[0, 0])
    o2 = oracle.Oracle(1, 2, 2, 4, 1, [0])
    o2.layer_forward(0, None, k[:, :5], v[:, :5])
    np.testing.assert_array_equal(o2.layer_forward(0, q[:, 5], k[:, 5:], v[:, 5:]), out[:, 5])
    with pytest.raises(RuntimeError):
        o.layer_prefill(0, RNG.standard_normal((1, 7, 2, 4)))     # more queries than cached rows


# ---------------------------------------------------------------- eviction (intra-layer compression mechanics)
def _random_keep(rng, B, Hkv, n, lo_frac=0.5):
    n_keep = rng.integers(max(1, int(n * lo_frac)), n + 1, size=(B, Hkv)).astype(np.int32)
    keep = np.zeros((B, Hkv, n), dtype=np.int32)
    for b in range(B):
        for h in range(Hkv):
            keep[b, h, : n_keep[b, h]] = np.sort(rng.choice(n, size=n_keep[b, h], replace=False))
    return keep, n_keep


def test_eviction_against_brute_force_with_sharing_and_later_appends():
    """Layer 1's cache is sparsified; layer 3 shares it and must see exactly the kept rows (and the
    rows appended afterwards); layers 0 and 2 are untouched."""
    L, Hq, Hkv, D, B, ctx = 4, 4, 2, 8, 2, 12
    sm = [0, 1, 2, 1]
    rng = np.random.default_rng(77)
    o, kc, vc, qs, ks, vs, outs = run_oracle(L, Hq, Hkv, D, B, sm, ctx, 1, rng)
    keep, n_keep = _random_keep(rng, B, Hkv, ctx + 1)
    o.evict(1, keep, n_keep)
    q2 = rng.standard_normal((L, B, Hq, D))
    k2 = rng.standard_normal((L, B, 1, Hkv, D))
    v2 = rng.standard_normal((L, B, 1, Hkv, D))
    out2 = o.step(q2, k2, v2)
    G = Hq // Hkv
    for l in range(L):
        r = 1 if l == 3 else l
        Kfull = np.concatenate([kc[r], ks[0, r]], axis=1)         # [B][ctx+1][Hkv][D] before eviction
        Vfull = np.concatenate([vc[r], vs[0, r]], axis=1)
        for b in range(B):
            for hq in range(Hq):
                h = hq // G
                rows = keep[b, h, : n_keep[b, h]] if r == 1 else np.arange(ctx + 1)
                K = np.concatenate([Kfull[b, rows, h], k2[r, b, :, h]], axis=0)
                V = np.concatenate([Vfull[b, rows, h], v2[r, b, :, h]], axis=0)
                np.testing.assert_allclose(out2[l, b, hq], brute_attention(q2[l, b, hq], K, V), atol=1e-13)
                assert o.unit_len(l, b, h) == len(rows) + 1
    assert o.length(1) == int(n_keep.max()) + 1 and o.length(0) == ctx + 2


def test_removing_one_row_follows_the_softmax_removal_identity():
    """out' = (out * Z - e_j v_j) / (Z - e_j): dropping row j removes its term from both sums."""
    n, D = 9, 8
    q, K, V = RNG.standard_normal(D), RNG.standard_normal((n, D)), RNG.standard_normal((n, D))
    o = oracle.Oracle(1, 1, 1, D, 1, [0])
    o.layer_forward(0, None, K[None, :, None], V[None, :, None])
    full = o.layer_forward(0, q[None, None])[0, 0]
    j = 4
    rows = np.array([[[r for r in range(n) if r != j] + [0]]], dtype=np.int32)
    o.evict(0, rows, [[n - 1]])
    got = o.layer_forward(0, q[None, None])[0, 0]
    sc = K @ q / np.sqrt(D)
    e = np.exp(sc - sc.max())
    ref = (full * e.sum() - e[j] * V[j]) / (e.sum() - e[j])
    np.testing.assert_allclose(got, ref, atol=1e-13)


def test_keeping_everything_changes_nothing_and_bad_lists_are_rejected():
    L, Hq, Hkv, D, B = 2, 2, 2, 4, 1
    rng = np.random.default_rng(5)
    o, *_ = run_oracle(L, Hq, Hkv, D, B, [0, 0], 5, 1, rng)
    K0, V0 = o.cache(0)
    o.evict(0, np.tile(np.arange(6, dtype=np.int32), (B, Hkv, 1)), np.full((B, Hkv), 6))
    K1, V1 = o.cache(0)
    np.testing.assert_array_equal(K0, K1)
    np.testing.assert_array_equal(V0, V1)
    for bad_keep, bad_n in (([[[3, 2, 0, 0, 0, 0]] * 2], [[2, 2]]),      # not ascending
                            ([[[0, 6, 0, 0, 0, 0]] * 2], [[2, 2]]),      # out of range
                            ([[[0, 1, 2, 3, 4, 5]] * 2], [[0, 1]])):     # empty unit
        with pytest.raises(RuntimeError):
            o.evict(0, bad_keep, bad_n)
    with pytest.raises(RuntimeError):
        o.evict(1, np.zeros((B, Hkv, 6), dtype=np.int32), np.ones((B, Hkv)))     # layer 1 shares
    # prefill positions are undefined once units differ in length
    o.evict(0, [[[0, 1, 2, 0, 0, 0], [0, 1, 0, 0, 0, 0]]], [[3, 2]])
    with pytest.raises(RuntimeError):
        o.layer_prefill(0, rng.standard_normal((B, 1, Hq, D)))


# ---------------------------------------------------------------- strategy-search reductions
def test_layer_distances_against_numpy_and_metric_properties():
    L, Hq, Hkv, D, B, n = 5, 2, 2, 4, 6, 7
    rng = np.random.default_rng(13)
    o = oracle.Oracle(L, Hq, Hkv, D, B, np.arange(L))
    ks = rng.standard_normal((L, B, n, Hkv, D))
    vs = rng.standard_normal((L, B, n, Hkv, D))
    ks[3], vs[3] = ks[1], vs[1]                       # two identical layers
    ks[4], vs[4] = 2.0 * ks[0], 2.0 * vs[0]           # one layer is twice another
    for l in range(L):
        o.layer_forward(l, None, ks[l], vs[l])
    d = o.layer_distances()
    rep = np.concatenate([ks.mean(axis=1).reshape(L, -1), vs.mean(axis=1).reshape(L, -1)], axis=1)
    ref = np.linalg.norm(rep[:, None, :] - rep[None, :, :], axis=2)
    np.testing.assert_allclose(d, ref, atol=1e-12)
    assert np.all(np.diag(d) == 0) and np.array_equal(d, d.T) and d[1, 3] == 0
    assert d[0, 4] == pytest.approx(np.linalg.norm(rep[0]), abs=1e-12)            # |2x - x| = |x|
    for i in range(L):
        for j in range(L):
            for k in range(L):
                assert d[i, j] <= d[i, k] + d[k, j] + 1e-12
    # the mean is over sequences: permuting them changes nothing
    o2 = oracle.Oracle(L, Hq, Hkv, D, B, np.arange(L))
    perm = rng.permutation(B)
    for l in range(L):
        o2.layer_forward(l, None, ks[l][perm], vs[l][perm])
    np.testing.assert_allclose(o2.layer_distances(), d, atol=1e-12)


def test_layer_distances_need_equal_unevicted_caches():
    o = oracle.Oracle(2, 1, 1, 4, 1, [0, 1])
    o.layer_forward(0, None, RNG.standard_normal((1, 3, 1, 4)), RNG.standard_normal((1, 3, 1, 4)))
    with pytest.raises(RuntimeError):
        o.layer_distances()                           # layer 1 is empty


def test_mean_cosine_against_numpy_and_closed_forms():
    rng = np.random.default_rng(17)
    a, b = rng.standard_normal((5, 33)), rng.standard_normal((5, 33))
    ma, mb = a.mean(0), b.mean(0)
    assert oracle.mean_cosine(a, b) == pytest.approx(ma @ mb / np.linalg.norm(ma) / np.linalg.norm(mb), abs=1e-14)
    assert oracle.mean_cosine(a, a) == pytest.approx(1.0, abs=1e-14)
    assert oracle.mean_cosine(a, -3.0 * a) == pytest.approx(-1.0, abs=1e-14)
    assert oracle.mean_cosine(a, 7.5 * b) == pytest.approx(oracle.mean_cosine(a, b), abs=1e-14)
    e0, e1 = np.zeros((2, 4)), np.zeros((2, 4))
    e0[:, 0], e1[:, 1] = 1.0, 1.0
    assert oracle.mean_cosine(e0, e1) == 0.0
    # only the mean matters: sentences whose deviations cancel do not change the result
    dev = rng.standard_normal((1, 33))
    a2 = np.concatenate([a + dev, a - dev])
    b2 = np.concatenate([b, b])
    assert oracle.mean_cosine(a2, b2) == pytest.approx(oracle.mean_cosine(a, b), abs=1e-13)
