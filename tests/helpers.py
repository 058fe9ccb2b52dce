"""Shared plumbing of the GPU parity tests: feed the same seeded tensors to the CUDA
library (through its C ABI) and to the fp64 oracle, and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import synth_inputs as si
from paper_2410_18517_b200 import SharedKVCache

# Tolerances fixed by the build's target: bf16/fp32 inputs, fp32 accumulation.
MAX_ABS = 2e-3
REL_L2 = 1e-3


def assert_close(got: np.ndarray, ref: np.ndarray, what=""):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref).max()
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    assert err <= MAX_ABS, f"{what}: max-abs {err:.3e} > {MAX_ABS}"
    assert rel <= REL_L2, f"{what}: rel-L2 {rel:.3e} > {REL_L2}"
    return err, rel


GUARD_BYTES = 1 << 16
CANARY = 0xA5


class GuardedCache(SharedKVCache):
    """A cache whose pool and workspace sit between guard zones filled with a pattern, and whose
    rows that no token may ever occupy (rows max_seq .. row_stride-1 of every (sequence, head) unit,
    and whole units beyond the batch in use) are filled with the same pattern after binding.
    `check_canaries` verifies that no kernel wrote to any of them."""

    def _allocate(self, nbytes):
        big = self._torch.full((nbytes + 2 * GUARD_BYTES,), CANARY, dtype=self._torch.uint8, device=self.device)
        self.__dict__.setdefault("_guarded", []).append(big)
        return big[GUARD_BYTES:GUARD_BYTES + nbytes]

    def paint(self, max_seq, batch_in_use):
        self._max_seq, self._batch_in_use = max_seq, batch_in_use
        for s in range(self.num_slots()):
            for kv in (0, 1):
                p = self.plane(s, kv).view(self._torch.uint8)
                p[:, :, max_seq:] = CANARY
                p[batch_in_use:] = CANARY

    def check_canaries(self):
        torch_ = self._torch
        for big in self._guarded[:1]:      # the pool (the workspace is scratch the kernels may write anywhere in)
            assert bool((big[:GUARD_BYTES] == CANARY).all()) and bool((big[-GUARD_BYTES:] == CANARY).all()), "guard zone hit"
        for big in self._guarded[1:]:
            assert bool((big[:GUARD_BYTES] == CANARY).all()) and bool((big[-GUARD_BYTES:] == CANARY).all()), "workspace guard hit"
        for s in range(self.num_slots()):
            for kv in (0, 1):
                p = self.plane(s, kv).view(torch_.uint8)
                assert bool((p[:, :, self._max_seq:] == CANARY).all()), f"padding rows of plane ({s},{kv}) written"
                assert bool((p[self._batch_in_use:] == CANARY).all()), f"unused units of plane ({s},{kv}) written"


CACHE_CLASS = SharedKVCache       # the bounds-checking driver swaps in GuardedCache


def make_cache(w: si.Workload, extra_rows: int, share_map=None, device=0, scale=0.0, max_batch=None) -> SharedKVCache:
    sm = w.share_map() if share_map is None else share_map
    cache = CACHE_CLASS(w.L, w.Hq, w.Hkv, w.D, max_batch or w.B, w.context + extra_rows, w.dtype, share_map=sm,
                        softmax_scale=scale, device=device)
    if isinstance(cache, GuardedCache):
        cache.paint(w.context + extra_rows, w.B)
    return cache


def run_small(w: si.Workload, steps: int, share_map=None, options=(), check_cache=True, scale=None, use_step=False):
    """Whole-workload comparison: context load, then `steps` decode steps, every output and
    (optionally) every cached bit compared.  Inputs are generated on the CPU and copied.  With
    `use_step` a decode step goes through kvs_decode_step instead of kvs_append + kvs_decode_attention."""
    sm = np.asarray(w.share_map() if share_map is None else share_map)
    cache = make_cache(w, steps, sm, scale=0.0 if scale is None else scale)
    for opt, val in options:
        cache.set_option(opt, val)
    orc = oracle.Oracle(w.L, w.Hq, w.Hkv, w.D, w.B, sm, scale=scale)
    dev = cache.device
    for l in range(w.L):
        if w.context == 0:
            break
        k, v = si.context_kv(w, l)
        orc.layer_forward(l, None, k.double().numpy(), v.double().numpy())
        cache.append(l, k.to(dev), v.to(dev))
    worst = (0.0, 0.0)
    for t in range(steps):
        for l in range(w.L):
            q, k, v = si.step_qkv(w, t, l)
            ref = orc.layer_forward(l, q.double().numpy(), k.double().numpy(), v.double().numpy())
            if use_step:
                own = sm[l] == l
                out = cache.decode_step(l, q.to(dev), k.to(dev) if own else None, v.to(dev) if own else None)
            else:
                cache.append(l, k.to(dev), v.to(dev))
                out = cache.decode_attention(l, q.to(dev))
            e = assert_close(out.cpu().numpy(), ref, f"{w.name} step {t} layer {l}")
            worst = (max(worst[0], e[0]), max(worst[1], e[1]))
            assert cache.seq_len(l) == orc.length(l)
    assert cache.device_status() == 0
    if check_cache:
        _, root, slot = oracle.slot_table(sm)
        for l in range(w.L):
            n = orc.length(l)
            K, V = orc.cache(l)
            s = cache.slot_of_layer(l)
            assert s == slot[l]
            gk = cache.plane(s, 0)[: w.B, :, :n].double().cpu().numpy()
            gv = cache.plane(s, 1)[: w.B, :, :n].double().cpu().numpy()
            assert np.array_equal(gk, K) and np.array_equal(gv, V), f"cache bits differ, layer {l}"
    return cache, orc, worst


class SampledRun:
    """Full-size workload on the GPU with the oracle run on sampled (layer, b, q-head) units.

    Inputs are generated on the GPU (seeded), handed to the library, and the rows of the
    sampled units are sliced out of those same input tensors and copied to the host for
    the oracle -- the oracle never sees anything the library produced.
    """

    def __init__(self, w: si.Workload, steps: int, n_samples: int = 64, seed: int = 0, device: int = 0):
        self.w, self.steps = w, steps
        self.sm = w.share_map()
        _, self.root, _ = oracle.slot_table(self.sm)
        self.cache = make_cache(w, steps, self.sm, device)
        rng = np.random.default_rng(seed)
        sharing = [l for l in range(w.L) if self.sm[l] != l]
        layers = sharing + [int(x) for x in rng.integers(0, w.L, size=max(n_samples - len(sharing), 0))]
        self.samples = [(l, int(rng.integers(0, w.B)), int(rng.integers(0, w.Hq))) for l in layers]
        # rows of the (root layer, b, kv-head) units the samples read
        self.rows = {(int(self.root[l]), b, hq // w.G): ([], []) for (l, b, hq) in self.samples}

    def _keep(self, layer, k, v):
        for (r, b, hk), (ks, vs) in self.rows.items():
            if r == layer:
                ks.append(k[b, :, hk].double().cpu().numpy())
                vs.append(v[b, :, hk].double().cpu().numpy())

    def load_context(self):
        w, dev = self.w, self.cache.device
        for l in range(w.L):
            if self.sm[l] != l:
                self.cache.append(l, None, None, w.B, w.context)
                continue
            k, v = si.context_kv(w, l, device=dev)
            self.cache.append(l, k, v)
            self._keep(l, k, v)
            del k, v
        torch.cuda.synchronize(dev)

    def step(self, t: int, check: bool):
        """Run decode step t; if `check`, compare the sampled units.  Returns worst (max-abs, rel-L2)."""
        w, dev = self.w, self.cache.device
        outs, qs = {}, {}
        for l in range(w.L):
            q, k, v = si.step_qkv(w, t, l, device=dev)
            self.cache.append(l, k, v)
            if self.sm[l] == l:
                self._keep(l, k, v)
            out = self.cache.decode_attention(l, q)
            if check:
                for (sl, b, hq) in self.samples:
                    if sl == l:
                        outs[(l, b, hq)] = out[b, hq].cpu().numpy()
                        qs[(l, b, hq)] = q[b, hq].double().cpu().numpy()
        worst = (0.0, 0.0)
        if check:
            torch.cuda.synchronize(dev)
            n = w.context + t + 1
            for (l, b, hq) in self.samples:
                ks, vs = self.rows[(int(self.root[l]), b, hq // w.G)]
                K, V = np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)
                assert K.shape == (n, w.D) and self.cache.seq_len(l) == n
                ref = oracle.attend_unit(qs[(l, b, hq)], K, V)
                e = assert_close(outs[(l, b, hq)], ref, f"{w.name} step {t} unit {(l, b, hq)}")
                worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        return worst

    def check_cached_rows(self):
        """The rows of every sampled unit, context and appended, are in the pool bit for bit."""
        w = self.w
        for (r, b, hk), (ks, vs) in self.rows.items():
            K, V = np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)
            s = self.cache.slot_of_layer(r)
            gk = self.cache.plane(s, 0)[b, hk, : K.shape[0]].double().cpu().numpy()
            gv = self.cache.plane(s, 1)[b, hk, : V.shape[0]].double().cpu().numpy()
            assert np.array_equal(gk, K) and np.array_equal(gv, V), f"cached rows differ for unit {(r, b, hk)}"
