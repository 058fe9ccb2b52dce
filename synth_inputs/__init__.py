"""Seeded synthetic workloads for shared-KV decode attention.

This module holds input generators only: workload shapes, seeded share maps and
seeded N(0,1) tensors.  It contains none of the method's arithmetic and is the
one piece of code that both the CPU oracle's tests and the GPU library's tests
and benchmark draw on, so that both sides see the same bits.

The paper's workloads are real chat models run on real text (Llama2-7B/13B,
InternLM2, Mistral-7B; Section 4).  None of that data is used here: the shapes
(layers, heads, head size) stand in for those models and the values are
standard-normal draws.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    L: int          # transformer layers
    Hq: int         # query heads
    Hkv: int        # key/value heads
    D: int          # head size
    B: int          # sequences decoded together
    context: int    # cached tokens before the first decode step
    dtype: str      # storage type of Q/K/V: "f32" or "bf16"
    n_shared: int   # layers whose cache is replaced by an earlier layer's
    map_seed: int   # seed of the random share map (ignored if fixed_map is set)
    steps: int      # decode steps the workload asks for
    fixed_map: tuple | None = None

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def share_map(self) -> np.ndarray:
        if self.fixed_map is not None:
            return np.asarray(self.fixed_map, dtype=np.int32)
        return random_share_map(self.L, self.n_shared, self.map_seed)

    def kv_read_bytes_per_layer(self, n: int) -> int:
        """K and V rows of one layer's slot, each read once."""
        return 2 * self.B * self.Hkv * n * self.D * self.elem_bytes

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations the build is measured on.  "tiny" is checked whole
# against the oracle; the others are checked on sampled units.
WORKLOADS = {
    "tiny": Workload("tiny", L=4, Hq=4, Hkv=4, D=64, B=2, context=128, dtype="f32",
                     n_shared=1, map_seed=0, steps=9, fixed_map=(0, 1, 2, 1)),
    "7b_mha": Workload("7b_mha", L=32, Hq=32, Hkv=32, D=128, B=8, context=4096, dtype="bf16",
                       n_shared=8, map_seed=2, steps=20),
    # the 7B shape cut to 4 layers (2 GiB pool): small enough for profiler captures
    "7b_mha_l4": Workload("7b_mha_l4", L=4, Hq=32, Hkv=32, D=128, B=8, context=4096, dtype="bf16",
                          n_shared=1, map_seed=0, steps=20, fixed_map=(0, 1, 2, 1)),
    "gqa_long_l4": Workload("gqa_long_l4", L=4, Hq=32, Hkv=8, D=128, B=4, context=32768, dtype="bf16",
                            n_shared=1, map_seed=0, steps=20, fixed_map=(0, 1, 2, 1)),
    # the 13B shape cut to 3 layers and 4736 rows (3 GiB pool): the smallest launches (1.55 GB) that still take
    # the scalar kernel's long-launch geometry, for profiler captures of that kernel
    "13b_mha_l3": Workload("13b_mha_l3", L=3, Hq=40, Hkv=40, D=128, B=16, context=4736, dtype="bf16",
                           n_shared=1, map_seed=0, steps=20, fixed_map=(0, 1, 0)),
    "13b_mha": Workload("13b_mha", L=40, Hq=40, Hkv=40, D=128, B=16, context=8192, dtype="bf16",
                        n_shared=12, map_seed=3, steps=64),
    "gqa_long": Workload("gqa_long", L=32, Hq=32, Hkv=8, D=128, B=4, context=32768, dtype="bf16",
                         n_shared=10, map_seed=4, steps=20),
}

SWEEP_BATCH = (1, 8, 32, 64)
SWEEP_CONTEXT = (1024, 8192, 32768)
SWEEP_SHARED = (0, 4, 8, 10)   # 0 %, 12.5 %, 25 %, ~30 % of 32 layers


def sweep_points():
    """The 48 grouped-query sweep points, in a fixed order; seed = point index."""
    pts = []
    i = 0
    for B in SWEEP_BATCH:
        for n in SWEEP_CONTEXT:
            for P in SWEEP_SHARED:
                pts.append(Workload(f"sweep_b{B}_n{n}_p{P}", L=32, Hq=32, Hkv=8, D=128, B=B,
                                    context=n, dtype="bf16", n_shared=P, map_seed=i, steps=20))
                i += 1
    return pts


def workload_by_name(name: str) -> Workload:
    """A named configuration, or a sweep point by its name (``sweep_b32_n8192_p10``)."""
    if name in WORKLOADS:
        return WORKLOADS[name]
    for w in sweep_points():
        if w.name == name:
            return w
    raise KeyError(f"unknown workload {name!r}")


def random_share_map(L: int, n_shared: int, seed: int) -> np.ndarray:
    """A random strategy with ``n_shared`` replaced layers.

    Stands in for the paper's randomly chosen strategies (Section 5, random
    sharing).  Draw the set T of replaced layers from {1..L-1}; then, in
    ascending order, give each its source uniformly among earlier layers that
    are not in T and not yet used as a source (so every source is a distinct
    layer that computes its own cache).  If some layer has no candidate left,
    draw everything again.
    """
    if not (0 <= n_shared <= (L // 2 if L > 1 else 0)):
        raise ValueError("n_shared must leave a distinct earlier source for every replaced layer")
    rng = np.random.default_rng(seed)
    while True:
        share_map = np.arange(L, dtype=np.int32)
        if n_shared == 0:
            return share_map
        targets = np.sort(rng.choice(np.arange(1, L), size=n_shared, replace=False))
        tset = set(int(t) for t in targets)
        used: set[int] = set()
        ok = True
        for t in targets:
            cand = [s for s in range(int(t)) if s not in tset and s not in used]
            if not cand:
                ok = False
                break
            s = int(rng.choice(cand))
            used.add(s)
            share_map[int(t)] = s
        if ok:
            return share_map


def _seed(*parts) -> int:
    h = hashlib.blake2b("/".join(str(p) for p in parts).encode(), digest_size=8).digest()
    return int.from_bytes(h, "little") & ((1 << 62) - 1)


def normal(parts: tuple, shape, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """N(0,1) draws (made in fp32, then rounded to ``dtype``) from a seed derived from ``parts``.

    The same ``parts`` on the same device type give the same bits.  CPU and CUDA
    generators differ, so a tensor is generated once and the very same tensor
    (moved or sliced with torch) is handed to both sides of a comparison.
    """
    g = torch.Generator(device=device)
    g.manual_seed(_seed(*parts))
    x = torch.randn(tuple(shape), generator=g, device=device, dtype=torch.float32)
    return x.to(dtype)


def context_kv(w: Workload, layer: int, device="cpu", base_seed: int = 0):
    """The context rows of one layer: (k, v), each ``[B][context][Hkv][D]``."""
    shape = (w.B, w.context, w.Hkv, w.D)
    k = normal((base_seed, w.name, "ctx_k", layer), shape, w.torch_dtype, device)
    v = normal((base_seed, w.name, "ctx_v", layer), shape, w.torch_dtype, device)
    return k, v


def step_qkv(w: Workload, step: int, layer: int, device="cpu", base_seed: int = 0):
    """One decode step's inputs of one layer: q ``[B][Hq][D]``, k/v ``[B][1][Hkv][D]``."""
    q = normal((base_seed, w.name, "q", step, layer), (w.B, w.Hq, w.D), w.torch_dtype, device)
    k = normal((base_seed, w.name, "k", step, layer), (w.B, 1, w.Hkv, w.D), w.torch_dtype, device)
    v = normal((base_seed, w.name, "v", step, layer), (w.B, 1, w.Hkv, w.D), w.torch_dtype, device)
    return q, k, v


def shard_batch(B: int, world_size: int, rank: int) -> tuple[int, int]:
    """Contiguous [start, stop) slice of the batch that ``rank`` decodes.

    Sequences are independent, so ranks share nothing on the data path.
    """
    base, rem = divmod(B, world_size)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)
